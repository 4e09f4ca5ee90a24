"""Pins for the oracle's segment planner (CPU only): hand-worked plans, an
O(T^2) selection written independently, numpy's stable argsort, and the
counting invariants of a stable grouping."""
import numpy as np
import pytest

from oracle import oracle
from paper_2605_13779_b200 import synth
from golden_io import read_golden


def brute_force_plan(keys):
    """keys[p] < 0 = dropped.  Repeatedly select the smallest remaining
    (key, index): quadratic, obviously the stable grouping."""
    remaining = [(int(k), p) for p, k in enumerate(keys) if k >= 0]
    perm, seg_key, seg_start = [], [], []
    while remaining:
        best = min(remaining)
        remaining.remove(best)
        if not seg_key or seg_key[-1] != best[0]:
            seg_key.append(best[0])
            seg_start.append(len(perm))
        perm.append(best[1])
    seg_start.append(len(perm))
    return np.array(perm, np.int32), np.array(seg_key, np.int32), np.array(seg_start, np.int32)


def keys_of(ids, table, num_slots, expert_ids=None):
    ids = np.asarray(ids)
    ok = (ids >= 0) & (ids < table.shape[0])
    slot = np.where(ok, table[np.clip(ids, 0, table.shape[0] - 1)], -1)
    if expert_ids is None:
        return slot
    K = expert_ids.shape[1]
    ps = np.repeat(slot, K)
    return np.where(ps >= 0, expert_ids.reshape(-1).astype(np.int64) * num_slots + ps, -1)


def check_invariants(plan, keys):
    keys = np.asarray(keys)
    active = np.nonzero(keys >= 0)[0]
    perm, seg_key, seg_start = plan["perm"], plan["seg_key"], plan["seg_start"]
    assert plan["n_active"] == active.size == perm.size
    assert sorted(perm.tolist()) == active.tolist()                  # a permutation of the active set
    assert seg_start[0] == 0 and seg_start[-1] == perm.size
    assert (np.diff(seg_key) > 0).all()                              # keys strictly increasing
    lens = np.diff(seg_start)
    assert (lens > 0).all() and lens.sum() == active.size
    counts = np.bincount(keys[active], minlength=1)
    np.testing.assert_array_equal(lens, counts[counts > 0])          # lengths = key histogram
    np.testing.assert_array_equal(seg_key, np.nonzero(counts)[0])
    for s in range(plan["S"]):
        seg = perm[seg_start[s]:seg_start[s + 1]]
        assert (keys[seg] == seg_key[s]).all()
        assert (np.diff(seg) > 0).all()                              # indices increasing inside a segment


def test_golden_plans():
    g = read_golden("plan_tiny.txt")
    p = oracle.plan(g["dense_ids"].astype(np.int64), g["dense_id_to_slot"].astype(np.int32),
                    int(g["dense_num_slots"][0]))
    np.testing.assert_array_equal(p["perm"], g["dense_perm"].astype(np.int32))
    np.testing.assert_array_equal(p["seg_key"], g["dense_seg_key"].astype(np.int32))
    np.testing.assert_array_equal(p["seg_start"], g["dense_seg_start"].astype(np.int32))
    assert p["n_not_resident"] == 0
    ns, ne = int(g["moe_num_slots"][0]), int(g["moe_num_experts"][0])
    p = oracle.plan(g["moe_ids"].astype(np.int64), np.arange(ns, dtype=np.int32), ns,
                    expert_ids=g["moe_experts"].astype(np.int32).reshape(3, 2), num_experts=ne)
    np.testing.assert_array_equal(p["perm"], g["moe_perm"].astype(np.int32))
    np.testing.assert_array_equal(p["seg_key"], g["moe_seg_key"].astype(np.int32))
    np.testing.assert_array_equal(p["seg_start"], g["moe_seg_start"].astype(np.int32))


@pytest.mark.parametrize("T,num_slots,p_none", [(0, 4, 0.0), (1, 1, 0.0), (7, 3, 0.5), (64, 4, 0.1),
                                                 (61, 64, 0.0), (50, 5, 1.0)])
def test_dense_plan_matches_brute_force(T, num_slots, p_none):
    rng = synth.stream("plan/brute", T, num_slots)
    ids = rng.integers(0, num_slots, size=T).astype(np.int64)
    ids[rng.random(T) < p_none] = -1
    table = rng.permutation(num_slots).astype(np.int32)
    p = oracle.plan(ids, table, num_slots)
    keys = keys_of(ids, table, num_slots)
    perm, seg_key, seg_start = brute_force_plan(keys)
    np.testing.assert_array_equal(p["perm"], perm)
    np.testing.assert_array_equal(p["seg_key"], seg_key)
    np.testing.assert_array_equal(p["seg_start"], seg_start)
    check_invariants(p, keys)


def test_moe_plan_matches_brute_force_and_argsort():
    batch = synth.config4_batch(T=24, E=6, K=3, num_slots=4, rank=2, p_none=0.2, tag="plan/moe")
    p = oracle.plan(batch.ids, batch.table.id_to_slot, 4, expert_ids=batch.expert_ids, num_experts=6)
    keys = keys_of(batch.ids, batch.table.id_to_slot, 4, batch.expert_ids)
    perm, seg_key, seg_start = brute_force_plan(keys)
    np.testing.assert_array_equal(p["perm"], perm)
    np.testing.assert_array_equal(p["seg_key"], seg_key)
    np.testing.assert_array_equal(p["seg_start"], seg_start)
    check_invariants(p, keys)


@pytest.mark.parametrize("which", ["config2", "config3", "config5", "config4"])
def test_plan_equals_numpy_stable_argsort_on_benchmark_batches(which):
    expert_ids, E = None, 0
    if which == "config2":
        b = synth.config2_batch()
        ids, table = b.ids, b.table
    elif which == "config3":
        b = synth.config3_batch(bijection=False)
        ids, table = b.ids, b.table
    elif which == "config5":
        c = synth.config5(d=8, n=8)
        ids, table = c.ids, c.table
    else:
        b = synth.config4_batch(T=512)
        ids, table, expert_ids, E = b.ids, b.table, b.expert_ids, b.E
    p = oracle.plan(ids, table.id_to_slot, table.num_slots, expert_ids=expert_ids, num_experts=E)
    keys = keys_of(ids, table.id_to_slot, table.num_slots, expert_ids)
    active = np.nonzero(keys >= 0)[0]
    order = active[np.argsort(keys[active], kind="stable")]
    np.testing.assert_array_equal(p["perm"], order.astype(np.int32))
    check_invariants(p, keys)


def test_non_resident_tokens_are_dropped_and_counted():
    table = np.array([0, -1, 1, 7], dtype=np.int32)      # id 3 maps outside a 2-slot pool
    ids = np.array([0, 1, 2, 3, 99, -1, -5, 2], dtype=np.int64)
    p = oracle.plan(ids, table, 2)
    np.testing.assert_array_equal(p["perm"], [0, 2, 7])
    np.testing.assert_array_equal(p["seg_key"], [0, 1])
    np.testing.assert_array_equal(p["seg_start"], [0, 1, 3])
    assert p["n_not_resident"] == 4                      # ids 1, 3, 99, -5

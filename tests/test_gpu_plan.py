"""Segment plans from the CUDA planner are bit-exact against the oracle's."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2605_13779_b200 import synth

pytestmark = pytest.mark.gpu


def gpu_plan(ids, table_np, expert_ids=None, num_experts=0):
    from paper_2605_13779_b200 import binding as mb, harness
    table = harness.upload_table(table_np)
    ids_d = torch.from_numpy(np.ascontiguousarray(ids, dtype=np.int64)).cuda()
    ex_d = None
    if expert_ids is not None:
        ex_d = torch.from_numpy(np.ascontiguousarray(expert_ids, dtype=np.int32)).cuda()
    status = mb.new_status()
    plan = mb.mint_lora_plan(table, ids_d, status, expert_ids=ex_d, num_experts=num_experts)
    return plan.arrays(), status.cpu().numpy()


def check(ids, table_np, expert_ids=None, num_experts=0):
    got, status = gpu_plan(ids, table_np, expert_ids, num_experts)
    ref = oracle.plan(ids, table_np.id_to_slot, table_np.num_slots, expert_ids=expert_ids,
                      num_experts=num_experts)
    assert got["S"] == ref["S"] and got["n_active"] == ref["n_active"]
    np.testing.assert_array_equal(got["perm"], ref["perm"])
    np.testing.assert_array_equal(got["seg_start"], ref["seg_start"])
    np.testing.assert_array_equal(got["seg_key"], ref["seg_key"])
    assert got["n_not_resident"] == ref["n_not_resident"]
    assert got["n_bad_expert"] == ref["n_bad_expert"]
    if ref["S"]:
        assert got["max_segment"] == int(np.diff(ref["seg_start"]).max())
    return got, ref, status


def test_config1_plan():
    c = synth.config1()
    got, ref, status = check(c.ids, c.table)
    assert status[0] == 0 and got["n_active"] < c.T       # some tokens have no adapter


def test_config2_plan():
    b = synth.config2_batch()
    got, _, status = check(b.ids, b.table)
    assert status[0] == 0
    slots = np.unique(b.ids)
    assert got["sum_rank"] == int(b.table.slot_rank[slots].sum())


@pytest.mark.parametrize("bijection", [True, False])
def test_config3_plan(bijection):
    b = synth.config3_batch(bijection=bijection)
    check(b.ids, b.table)


def test_config4_plan_full_size():
    b = synth.config4_batch()
    got, ref, _ = check(b.ids, b.table, b.expert_ids, b.E)
    assert got["n_active"] == 4096 * 8 and got["S"] > 1900


def test_config5_plan_million_id_catalog():
    c = synth.config5(d=8, n=8)
    got, ref, status = check(c.ids, c.table)
    assert status[0] == 0 and got["S"] == c.meta["distinct"]


@pytest.mark.parametrize("T,num_slots,p_none", [(0, 4, 0.0), (1, 1, 0.0), (5, 3, 1.0), (31, 2, 0.3),
                                                 (32, 2, 0.0), (33, 700, 0.1), (1023, 5, 0.2),
                                                 (1024, 64, 0.0), (1025, 300, 0.5), (4097, 4096, 0.05),
                                                 (20000, 3, 0.01), (40000, 70000, 0.1)])
def test_random_dense_plans(T, num_slots, p_none):
    rng = synth.stream("gpu/plan", T, num_slots)
    ids = rng.integers(0, num_slots, size=T).astype(np.int64)
    ids[rng.random(T) < p_none] = -1
    ranks = np.ones(num_slots, dtype=np.int32)
    table = synth.identity_table(num_slots, ranks)
    table.id_to_slot = rng.permutation(num_slots).astype(np.int32)
    check(ids, table)


@pytest.mark.parametrize("T,K,E,num_slots", [(7, 2, 3, 2), (100, 4, 8, 5), (513, 8, 128, 16), (64, 1, 1, 1),
                                              (300, 6, 60, 64)])
def test_random_moe_plans(T, K, E, num_slots):
    b = synth.config4_batch(T=T, E=E, K=K, num_slots=num_slots, rank=2, p_none=0.15, tag="gpu/moeplan")
    check(b.ids, b.table, b.expert_ids, E)


def test_non_resident_and_bad_expert_are_reported():
    from paper_2605_13779_b200 import binding as mb
    c = synth.config5(T=256, d=8, n=8, leave_unbound=3)
    got, ref, status = check(c.ids, c.table)
    assert ref["n_not_resident"] > 0
    assert status[0] == mb.MINT_ERR_NOT_RESIDENT and status[1] == ref["n_not_resident"]
    first = int(np.nonzero(c.table.id_to_slot[c.ids] < 0)[0][0])
    assert status[2] == first
    # ids outside the catalog are not resident either
    ids = np.array([0, 5, 123456789, -7, 1], dtype=np.int64)
    table = synth.identity_table(4, np.ones(4, np.int32))
    got, ref, status = check(ids, table)
    assert got["n_not_resident"] == 3 and status[0] == mb.MINT_ERR_NOT_RESIDENT
    # an expert id outside [0, E) drops the pair and reports BAD_INDEX
    b = synth.config4_batch(T=16, E=4, K=2, num_slots=2, rank=1, tag="gpu/badexp")
    ex = b.expert_ids.copy()
    ex[3, 1] = 9
    got, ref, status = check(b.ids, b.table, ex, 4)
    assert got["n_bad_expert"] == 1 and status[0] == mb.MINT_ERR_BAD_INDEX and status[2] == 7


def test_plan_is_deterministic():
    b = synth.config4_batch(T=1024)
    a1, _ = gpu_plan(b.ids, b.table, b.expert_ids, b.E)
    a2, _ = gpu_plan(b.ids, b.table, b.expert_ids, b.E)
    for k in ("perm", "seg_start", "seg_key"):
        np.testing.assert_array_equal(a1[k], a2[k])


@pytest.mark.parametrize("T,K,E,num_slots", [(4096, 1, 0, 7), (5000, 1, 0, 4096), (18439, 1, 0, 32), (600, 8, 128, 16),
                                              (4096, 8, 128, 32), (1111, 6, 60, 64), (262144, 1, 0, 3)])
def test_plans_of_the_grid_wide_sort(T, K, E, num_slots):
    """Batches of 4096 .. 262 144 items over at most 4096 keys are sorted by the counting sort that
    runs on one CTA per 1024 items: tokens without an adapter, ids that are not resident, expert ids
    out of range, ranks 1 and above side by side, and a segment long enough for the dense tiles."""
    from paper_2605_13779_b200 import binding as mb
    rng = synth.stream("gpu/plan/grid", T, K, E, num_slots)
    ids = rng.integers(0, num_slots, size=T).astype(np.int64)
    ids[rng.random(T) < 0.3] = 0                       # one long segment
    ids[rng.random(T) < 0.05] = -1
    ranks = rng.choice(np.array([1, 8, 16], dtype=np.int32), size=num_slots)
    table = synth.identity_table(num_slots, ranks)
    table.id_to_slot = rng.permutation(num_slots).astype(np.int32)
    if num_slots > 4:
        table.id_to_slot[rng.integers(0, num_slots, size=2)] = -1      # two catalog ids without a slot
    ex = None
    if E:
        ex = np.stack([rng.permutation(E)[:K] for _ in range(T)]).astype(np.int32)
        ex[T // 3, K - 1] = E + 5
        ex[T // 2, 0] = -1
    got, ref, status = check(ids, table, ex, E)
    assert got["sum_rank"] == int(ranks[ref["seg_key"] % num_slots].sum())
    if ref["n_not_resident"]:
        assert status[0] == mb.MINT_ERR_NOT_RESIDENT and status[1] == ref["n_not_resident"]
        assert status[2] == int(np.nonzero((ids >= 0) & (table.id_to_slot[np.maximum(ids, 0)] < 0))[0][0])
    elif E:
        assert status[0] == mb.MINT_ERR_BAD_INDEX and got["n_bad_expert"] == 2

"""Backward of the MoE expert LoRA apply on the GPU against the fp64 oracle.

Tolerances as for the dense backward: dx (bf16, one row per pair, accumulated into) within
max |delta| <= 3e-2 and relative Frobenius <= 5e-3 over the full tensor and again from dx0 = 0;
dA, dB (fp32, packed per-expert tensors) relative Frobenius <= 1e-4 per (slot, expert) block on the
update itself; ranks at or above the slot's rank and blocks without pairs bit for bit."""
import numpy as np
import pytest
import torch

from oracle import backward
from paper_2605_13779_b200 import synth
import parity

pytestmark = pytest.mark.gpu


def run(case, dy, dx0_zero=False, weighted=True, want_dx=True, want_grads=True, expert_ids=None, repeat=1):
    from paper_2605_13779_b200 import binding as mb, harness
    dev = harness.upload_moe(case)
    P = case.T * case.K
    ex = dev.expert_ids if expert_ids is None else torch.from_numpy(np.ascontiguousarray(expert_ids)).cuda()
    dyd = mb.bf16_from_bits(dy)
    dx0 = np.zeros((P, case.d), np.uint16) if dx0_zero else synth.normal_bf16(synth.stream(case.name, "dx0"), (P, case.d), 1.0)
    dx = mb.bf16_from_bits(dx0) if want_dx else None
    dA0 = synth.stream(case.name, "dA0").standard_normal(case.A.shape).astype(np.float32)
    dB0 = synth.stream(case.name, "dB0").standard_normal(case.B.shape).astype(np.float32)
    dA = torch.from_numpy(dA0.copy()).cuda() if want_grads else None
    dB = torch.from_numpy(dB0.copy()).cuda() if want_grads else None
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status, expert_ids=ex, num_experts=case.E)
    for _ in range(repeat):
        mb.mint_moe_lora_backward(dev.pool, dev.table, plan, dev.x, dyd, dev.status, dx=dx, dA=dA, dB=dB,
                                  x_row=dev.x_row, pair_weight=dev.pair_weight if weighted else None)
    torch.cuda.synchronize()
    out = {"status": dev.status.cpu().numpy(), "dx0": dx0, "dA0": dA0, "dB0": dB0}
    if want_dx:
        out["dx"] = harness.y_to_f64(dx)
    if want_grads:
        out["dA"] = dA.cpu().numpy().astype(np.float64)
        out["dB"] = dB.cpu().numpy().astype(np.float64)
    return out


def reference(case, dy, dx0, dA0, dB0, weighted=True, expert_ids=None):
    t = case.table
    return backward.moe_lora_backward(case.ids, case.expert_ids if expert_ids is None else expert_ids, t.id_to_slot,
                                      t.slot_rank, t.slot_scale, case.A, case.B, case.x, dy, x_row=case.x_row,
                                      pair_weight=case.pair_weight if weighted else None, dx0=dx0, dA0=dA0, dB0=dB0)


def check_blocks(got, ref, start, rank_axis, case, what, expert_ids=None):
    """Per (slot, expert) block: the update within 1e-4 relative Frobenius, everything else bit for bit."""
    t = case.table
    ex = case.expert_ids if expert_ids is None else expert_ids
    used = np.zeros((t.num_slots, case.E), bool)
    for tt in np.nonzero(case.ids >= 0)[0]:
        slot = t.id_to_slot[case.ids[tt]]
        if slot >= 0:
            ok = (ex[tt] >= 0) & (ex[tt] < case.E)
            used[slot, ex[tt][ok]] = True
    start = start.astype(np.float64)
    for slot in range(t.num_slots):
        r = int(t.slot_rank[slot])
        np.testing.assert_array_equal(got[slot][~used[slot]], start[slot][~used[slot]], err_msg=f"{what}: idle blocks of slot {slot}")
        lo = [slice(None)] * 3
        hi = [slice(None)] * 3
        lo[rank_axis], hi[rank_axis] = slice(0, r), slice(r, None)
        g, f, s0 = got[slot][used[slot]], ref[slot][used[slot]], start[slot][used[slot]]
        np.testing.assert_array_equal(g[tuple(hi)], s0[tuple(hi)], err_msg=f"{what}: padding of slot {slot}")
        for b in range(g.shape[0]):
            d_ref = f[b][tuple(lo[1:])] - s0[b][tuple(lo[1:])]
            d_got = g[b][tuple(lo[1:])] - s0[b][tuple(lo[1:])]
            err, denom = np.linalg.norm(d_got - d_ref), np.linalg.norm(d_ref)
            ulp = 6e-8 * np.linalg.norm(f[b][tuple(lo[1:])])
            assert err <= 1e-4 * denom + 2 * ulp, f"{what}: slot {slot} block {b} rel {err / max(denom, 1e-30):.3e}"


def check_case(case, what, weighted=True, expert_ids=None):
    P = case.T * case.K
    dy = synth.normal_bf16(synth.stream(case.name, "dy"), (P, case.n), 1.0)
    for dx0_zero in (False, True):
        got = run(case, dy, dx0_zero=dx0_zero, weighted=weighted, expert_ids=expert_ids)
        dx, dA, dB, _ = reference(case, dy, got["dx0"], got["dA0"], got["dB0"], weighted=weighted, expert_ids=expert_ids)
        parity.assert_close(got["dx"], dx, f"{what}: dx (dx0 zero: {dx0_zero})")
        check_blocks(got["dA"], dA, got["dA0"], 2, case, f"{what}: dA", expert_ids)     # [E, d, r]: rank is the last axis
        check_blocks(got["dB"], dB, got["dB0"], 1, case, f"{what}: dB", expert_ids)     # [E, r, n]
    return got


@pytest.mark.parametrize("proj", ["gate", "down"])
@pytest.mark.parametrize("T,K,E,num_slots,rank,d,n", [(40, 4, 16, 5, 8, 264, 136), (512, 8, 128, 16, 16, 2048, 768),
                                                      (96, 2, 6, 3, 16, 520, 1032)])
def test_moe_backward_matches_oracle(proj, T, K, E, num_slots, rank, d, n):
    batch = synth.config4_batch(T=T, E=E, K=K, num_slots=num_slots, rank=rank, p_none=0.1, tag="gpu/moe-bwd")
    if proj == "down":
        d, n = n, d
    case = synth.config4_projection(batch, proj, d=d, n=n, tag="gpu/moe-bwd")
    got = check_case(case, f"moe backward {proj} T={T}")
    assert got["status"][0] == 0


def test_moe_backward_mixed_ranks_unweighted_and_bad_experts():
    """Slots of ranks 1, 3, 8 and 16 in a pool of r_max 16 (padding bit for bit), no routing weights,
    two expert ids out of range (their pairs keep their dx rows), tokens without an adapter."""
    from paper_2605_13779_b200 import binding as mb
    batch = synth.config4_batch(T=200, E=12, K=3, num_slots=4, rank=16, p_none=0.2, tag="gpu/moe-bwd/mixed")
    batch.table.slot_rank = np.array([1, 3, 8, 16], dtype=np.int32)
    case = synth.config4_projection(batch, "gate", d=392, n=264, tag="gpu/moe-bwd/mixed")
    ex = case.expert_ids.copy()
    live = np.nonzero(case.ids >= 0)[0]
    ex[live[0], 1] = 99
    ex[live[5], 0] = -2
    got = check_case(case, "moe backward mixed ranks", weighted=False, expert_ids=ex)
    assert got["status"][0] == mb.MINT_ERR_BAD_INDEX
    dead = np.repeat(case.ids < 0, case.K)
    dead[live[0] * case.K + 1] = dead[live[5] * case.K] = True
    np.testing.assert_array_equal(got["dx"][dead], synth.bf16_bits_to_f64(got["dx0"])[dead])


def test_moe_backward_parts_and_repeat():
    """dx alone, the weight gradients alone, and two calls in a row (gradient accumulation) on one workspace."""
    batch = synth.config4_batch(T=64, E=8, K=2, num_slots=3, rank=8, tag="gpu/moe-bwd/parts")
    case = synth.config4_projection(batch, "down", d=136, n=264, tag="gpu/moe-bwd/parts")
    P = case.T * case.K
    dy = synth.normal_bf16(synth.stream(case.name, "dy"), (P, case.n), 1.0)
    only_dx = run(case, dy, want_grads=False)
    only_g = run(case, dy, want_dx=False)
    both = run(case, dy)
    np.testing.assert_array_equal(only_dx["dx"], both["dx"])
    np.testing.assert_array_equal(only_g["dA"], both["dA"])
    np.testing.assert_array_equal(only_g["dB"], both["dB"])
    twice = run(case, dy, dx0_zero=True, repeat=2)
    _, dA1, dB1, _ = reference(case, dy, twice["dx0"], np.zeros_like(twice["dA0"]), np.zeros_like(twice["dB0"]))
    for name, one in (("dA", dA1), ("dB", dB1)):
        delta = twice[name] - twice[name + "0"]
        assert np.linalg.norm(delta - 2 * one) <= 1e-4 * np.linalg.norm(2 * one) + 1e-5 * np.linalg.norm(twice[name + "0"])

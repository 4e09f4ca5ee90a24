"""MoE expert LoRA apply on the GPU against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2605_13779_b200 import synth
import parity

pytestmark = pytest.mark.gpu


def run_moe(case, weighted=False, y0_bits=None):
    from paper_2605_13779_b200 import binding as mb, harness
    dev = harness.upload_moe(case)
    if y0_bits is not None:
        dev.y = mb.bf16_from_bits(y0_bits)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status, expert_ids=dev.expert_ids, num_experts=case.E)
    mb.mint_moe_lora_apply(dev.pool, dev.table, plan, dev.x, dev.y, dev.status, x_row=dev.x_row,
                           pair_weight=dev.pair_weight if weighted else None)
    torch.cuda.synchronize()
    return harness.y_to_f64(dev.y), dev.status.cpu().numpy()


def check_case(case, what):
    for weighted in (False, True):
        y_ref, _ = parity.oracle_moe(case, weighted=weighted)
        y, status = run_moe(case, weighted=weighted)
        assert status[0] == 0, status
        parity.assert_close(y, y_ref, f"{what} weighted={weighted}")
    zero = np.zeros_like(case.y0)
    y_ref0, _ = parity.oracle_moe(case, y0=zero)
    y0, _ = run_moe(case, y0_bits=zero)
    parity.assert_close(y0, y_ref0, what + " y0=0")
    none = np.repeat(case.ids < 0, case.K)
    if none.any():
        y, _ = run_moe(case)
        np.testing.assert_array_equal(y[none], synth.bf16_bits_to_f64(case.y0)[none])


@pytest.mark.parametrize("proj", ["gate", "down"])
def test_config4_reduced_tokens(proj):
    """30B-A3B shapes (hidden 2048, 128 experts, top-8, expert width 768, 16 rank-16
    adapters) at T=512 tokens: 4096 pairs in about 1750 (expert, adapter) groups."""
    batch = synth.config4_batch(T=512)
    check_case(synth.config4_projection(batch, proj), f"config4/{proj}/T512")


@pytest.mark.parametrize("proj", ["gate", "down"])
def test_config4_full_size(proj):
    """The 30B-A3B setting as the benchmark runs it: T=4096 tokens, 32 768 pairs in
    2048 (expert, adapter) groups of 16 pairs on average; unweighted, weighted and
    with y = 0."""
    batch = synth.config4_batch()
    assert batch.T == 4096
    check_case(synth.config4_projection(batch, proj), f"config4/{proj}/T4096")


def test_config4_contiguous_requests_fewer_experts():
    """Fewer experts and contiguous requests give long (expert, adapter) groups."""
    batch = synth.config4_batch(T=768, E=8, K=2, num_slots=4, rank=16, contiguous_requests=True,
                                tag="config4/long")
    check_case(synth.config4_projection(batch, "gate", tag="config4/long"), "config4/long")


@pytest.mark.parametrize("T,K,E,d,n,num_slots,rank,p_none", [
    (1, 1, 1, 8, 8, 1, 1, 0.0),
    (9, 2, 3, 72, 40, 2, 3, 0.2),
    (65, 4, 16, 520, 264, 5, 8, 0.1),
    (33, 8, 32, 256, 1024, 3, 24, 0.0),
    (40, 2, 4, 768, 2048, 2, 1, 0.0),
])
def test_ragged_moe(T, K, E, d, n, num_slots, rank, p_none):
    tag = f"gpu/moe/{T}/{K}/{E}"
    batch = synth.config4_batch(T=T, E=E, K=K, num_slots=num_slots, rank=rank, p_none=p_none, tag=tag)
    check_case(synth.config4_projection(batch, "gate", d=d, n=n, tag=tag), tag + "/gate")
    check_case(synth.config4_projection(batch, "down", d=d, n=n, tag=tag), tag + "/down")


@pytest.mark.parametrize("r_max,ranks,d,n", [
    (16, [16, 1, 9, 8], 520, 264),
    (32, [32, 3, 17, 8, 24], 2048, 768),
    (64, [64, 40, 1, 16, 33, 8], 776, 2048),
    (8, [8, 2, 5], 264, 136),
])
def test_mixed_ranks_in_padded_pools(r_max, ranks, d, n):
    """Slots of different ranks in one pool of r_max columns; the padding is NaN
    and must never reach y.  Long and short (expert, adapter) groups."""
    import dataclasses
    tag = f"gpu/moe/mixed/{r_max}"
    S = len(ranks)
    batch = synth.config4_batch(T=160, E=4, K=2, num_slots=S, rank=r_max, p_none=0.05, tag=tag)
    table = synth.identity_table(S, np.asarray(ranks, dtype=np.int32), 2.0)
    batch = dataclasses.replace(batch, table=table)
    for proj in ("gate", "down"):
        check_case(synth.config4_projection(batch, proj, d=d, n=n, tag=tag), f"{tag}/{proj}")


def test_one_expert_top1_equals_dense_apply():
    from paper_2605_13779_b200 import binding as mb, harness
    batch = synth.config4_batch(T=50, E=1, K=1, num_slots=3, rank=8, tag="gpu/moe1")
    case = synth.config4_projection(batch, "gate", d=256, n=128, tag="gpu/moe1")
    y_moe, status = run_moe(case)
    assert status[0] == 0
    A_rd = np.ascontiguousarray(case.A[:, 0].transpose(0, 2, 1))      # [slot][r][d]
    dense = synth.DenseCase("dense", case.T, case.d, case.n, case.r_max, case.table, case.ids, A_rd,
                            np.ascontiguousarray(case.B[:, 0]), case.x, case.y0)
    dev = harness.upload_dense(dense)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    mb.mint_lora_apply_fused(dev.pool, dev.table, plan, dev.x, dev.y, dev.status)
    y_dense = harness.y_to_f64(dev.y)
    assert np.abs(y_moe - y_dense).max() <= 2.0 ** -6


def test_bad_row_index_is_reported_and_skipped():
    from paper_2605_13779_b200 import binding as mb, harness
    batch = synth.config4_batch(T=8, E=2, K=2, num_slots=2, rank=2, tag="gpu/moebad")
    case = synth.config4_projection(batch, "gate", d=64, n=64, tag="gpu/moebad")
    dev = harness.upload_moe(case)
    rows = case.x_row.copy()
    rows[5] = 10_000
    x_row = torch.from_numpy(rows).cuda()
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status, expert_ids=dev.expert_ids, num_experts=case.E)
    mb.mint_moe_lora_apply(dev.pool, dev.table, plan, dev.x, dev.y, dev.status, x_row=x_row)
    torch.cuda.synchronize()
    status = dev.status.cpu().numpy()
    assert status[0] == mb.MINT_ERR_BAD_INDEX and status[2] == 5
    y = harness.y_to_f64(dev.y)
    np.testing.assert_array_equal(y[5], synth.bf16_bits_to_f64(case.y0)[5])
    y_ref, _ = parity.oracle_moe(case)
    keep = np.arange(16) != 5
    parity.assert_close(y[keep], y_ref[keep], "other pairs")


def run_combine(case, y0_bits):
    from paper_2605_13779_b200 import binding as mb, harness
    dev = harness.upload_moe(case)
    y = mb.bf16_from_bits(y0_bits)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status, expert_ids=dev.expert_ids, num_experts=case.E)
    mb.mint_moe_lora_apply_combine(dev.pool, dev.table, plan, dev.x, y, dev.status, dev.pair_weight, x_row=dev.x_row)
    torch.cuda.synchronize()
    return harness.y_to_f64(y), dev.status.cpu().numpy()


def check_combine(case, what):
    from oracle import oracle
    t = case.table
    for zero in (False, True):
        y0 = synth.normal_bf16(synth.stream(what, "y0 tokens"), (case.T, case.n), 1.0)
        if zero:
            y0 = np.zeros_like(y0)
        y_ref, _ = oracle.moe_lora_apply_combine(case.ids, case.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                                 case.A, case.B, case.x, y0, case.pair_weight, x_row=case.x_row)
        y, status = run_combine(case, y0)
        assert status[0] == 0, status
        parity.assert_close(y, y_ref, f"{what} combine zero={zero}")
        none = case.ids < 0
        if none.any():
            np.testing.assert_array_equal(y[none], synth.bf16_bits_to_f64(y0)[none])


def test_combine_config4_down_reduced_tokens():
    batch = synth.config4_batch(T=512)
    check_combine(synth.config4_projection(batch, "down"), "config4/down/T512")


def test_combine_config4_down_full_size():
    batch = synth.config4_batch()
    check_combine(synth.config4_projection(batch, "down"), "config4/down/T4096")


@pytest.mark.parametrize("T,K,E,d,n,num_slots,rank,p_none", [
    (1, 1, 1, 8, 8, 1, 1, 0.0),
    (9, 2, 3, 72, 40, 2, 3, 0.3),
    (65, 4, 16, 520, 264, 5, 8, 0.1),
    (33, 8, 32, 256, 1024, 3, 24, 0.0),
])
def test_combine_ragged(T, K, E, d, n, num_slots, rank, p_none):
    tag = f"gpu/moe/combine/{T}/{K}/{E}"
    batch = synth.config4_batch(T=T, E=E, K=K, num_slots=num_slots, rank=rank, p_none=p_none, tag=tag)
    check_combine(synth.config4_projection(batch, "down", d=d, n=n, tag=tag), tag)
    check_combine(synth.config4_projection(batch, "gate", d=d, n=n, tag=tag), tag + "/rows-of-tokens")


def test_combine_is_deterministic():
    batch = synth.config4_batch(T=256)
    case = synth.config4_projection(batch, "down")
    y0 = synth.normal_bf16(synth.stream("gpu/moe/combine/det"), (case.T, case.n), 1.0)
    a, _ = run_combine(case, y0)
    b, _ = run_combine(case, y0)
    np.testing.assert_array_equal(a, b)


# ---- grouped call: several projections over the same routed pairs in one launch pair ----
def run_moe_grouped(cases, weighted, y0_zero=False):
    from paper_2605_13779_b200 import binding as mb, harness
    table = harness.upload_table(cases[0].table)
    devs = [harness.upload_moe(c, table=table) for c in cases]
    for i in range(1, len(cases)):   # projections with the same hidden states read one tensor
        if cases[i].x.shape == cases[i - 1].x.shape and np.array_equal(cases[i].x, cases[i - 1].x):
            devs[i].x = devs[i - 1].x
    if y0_zero:
        for dv in devs:
            dv.y.zero_()
    d0 = devs[0]
    plan = mb.mint_lora_plan(table, d0.ids, d0.status, expert_ids=d0.expert_ids, num_experts=cases[0].E)
    ws = [mb.new_moe_workspace(dv.pool, plan.T, plan.K) for dv in devs]
    for w in ws:
        w.fill_(0xFF)   # the workspace needs no initialisation
    mb.mint_moe_lora_apply_grouped([(dv.pool, dv.x, dv.y, w) for dv, w in zip(devs, ws)], table, plan, d0.status,
                                   x_row=d0.x_row, pair_weight=d0.pair_weight if weighted else None)
    torch.cuda.synchronize()
    return [harness.y_to_f64(dv.y) for dv in devs], d0.status.cpu().numpy()


def check_grouped(cases, what):
    for weighted, y0_zero in ((False, False), (True, False), (False, True)):
        ys, status = run_moe_grouped(cases, weighted, y0_zero)
        assert status[0] == 0, status
        for c, y in zip(cases, ys):
            y_ref, _ = parity.oracle_moe(c, weighted=weighted, y0=np.zeros_like(c.y0) if y0_zero else None)
            parity.assert_close(y, y_ref, f"{what} {c.name} weighted={weighted} y0_zero={y0_zero}")


@pytest.mark.parametrize("T", [512, 4096])
def test_config4_gate_and_up_in_one_call(T):
    """Gate and up read the same hidden rows for the same routed pairs: one grouped call, as
    the benchmark issues it."""
    batch = synth.config4_batch(T=T)
    cases = [synth.config4_projection(batch, "gate"), synth.config4_projection(batch, "up")]
    assert not np.array_equal(cases[0].A, cases[1].A) and np.array_equal(cases[0].x, cases[1].x)
    check_grouped(cases, f"config4/gate+up/T{T}")


def test_grouped_moe_projections_of_different_widths():
    tag = "gpu/moe/grouped"
    batch = synth.config4_batch(T=96, E=8, K=2, num_slots=3, rank=8, p_none=0.1, tag=tag)
    cases = [synth.config4_projection(batch, "gate", d=520, n=264, tag=tag),
             synth.config4_projection(batch, "up", d=520, n=1024, tag=tag),
             synth.config4_projection(batch, "gate", d=520, n=72, tag=tag + "/third")]
    check_grouped(cases, tag)
    none = np.repeat(batch.ids < 0, batch.K)
    ys, _ = run_moe_grouped(cases, weighted=True)
    for c, y in zip(cases, ys):
        np.testing.assert_array_equal(y[none], synth.bf16_bits_to_f64(c.y0)[none])


@pytest.mark.parametrize("r_max,ranks", [(16, [16, 1, 9, 8]), (8, [8, 2, 5]), (32, [32, 3, 17])])
def test_grouped_gate_and_up_share_x_with_mixed_ranks(r_max, ranks):
    """Gate and up over the same hidden states with slots of different ranks in NaN-padded pools:
    pools of at most 16 ranks take one pass over x for both, wider ones one pass each."""
    import dataclasses
    tag = f"gpu/moe/grouped-mixed/{r_max}"
    S = len(ranks)
    batch = synth.config4_batch(T=160, E=4, K=2, num_slots=S, rank=r_max, p_none=0.05, tag=tag)
    batch = dataclasses.replace(batch, table=synth.identity_table(S, np.asarray(ranks, dtype=np.int32), 2.0))
    cases = [synth.config4_projection(batch, "gate", d=520, n=264, tag=tag),
             synth.config4_projection(batch, "up", d=520, n=136, tag=tag)]
    check_grouped(cases, tag)

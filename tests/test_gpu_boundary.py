"""Boundary behaviour that needs a device: slot-table binds and evictions,
stale plans, shape checks, slot admission.  No test faults the GPU: every bad
input is caught on the host or skipped by the kernel's own checks."""
import numpy as np
import pytest
import torch

from paper_2605_13779_b200 import synth
import parity

pytestmark = pytest.mark.gpu


def test_bind_evict_and_generation():
    from paper_2605_13779_b200 import binding as mb
    t = mb.SlotTable(100, 4)
    g0 = t.generation
    t.bind(17, 2, 8, 2.0)
    t.bind(5, 0, 1, 0.5)
    assert t.generation == g0 + 2
    torch.cuda.synchronize()
    assert t.id_to_slot[17].item() == 2 and t.id_to_slot[5].item() == 0 and t.id_to_slot[6].item() == -1
    assert t.slot_rank.tolist() == [1, 0, 8, 0] and t.slot_scale.tolist() == [0.5, 0.0, 2.0, 0.0]
    with pytest.raises(mb.MintError) as e:
        t.bind(17, 1, 8, 2.0)            # id already resident
    assert e.value.status == mb.MINT_ERR_INVALID_ARG
    with pytest.raises(mb.MintError):
        t.bind(18, 2, 8, 2.0)            # slot occupied
    with pytest.raises(mb.MintError):
        t.bind(100, 1, 8, 2.0)           # outside the catalog
    with pytest.raises(mb.MintError) as e:
        t.bind(19, 1, 4096, 2.0)
    assert e.value.status == mb.MINT_ERR_RANK_TOO_LARGE
    with pytest.raises(mb.MintError) as e:
        t.evict(50)
    assert e.value.status == mb.MINT_ERR_NOT_RESIDENT
    t.evict(17)
    t.bind(18, 2, 4, 1.0)
    torch.cuda.synchronize()
    assert t.id_to_slot[17].item() == -1 and t.id_to_slot[18].item() == 2 and t.slot_rank[2].item() == 4


def test_stale_plan_is_refused_on_the_device():
    from paper_2605_13779_b200 import binding as mb, harness
    case = synth.random_dense_case("gpu/stale", 16, 64, 64, 3, [2, 2, 2], 2, p_none=0.0)
    dev = harness.upload_dense(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    dev.table.evict(1)                   # the table changes after the plan was made
    mb.mint_lora_apply_fused(dev.pool, dev.table, plan, dev.x, dev.y, dev.status)
    torch.cuda.synchronize()
    assert dev.status[0].item() == mb.MINT_ERR_STALE_PLAN
    np.testing.assert_array_equal(mb.bits_from_bf16(dev.y), case.y0)     # nothing was applied


def test_plan_for_another_batch_size_is_refused():
    from paper_2605_13779_b200 import binding as mb, harness
    case = synth.random_dense_case("gpu/shape", 16, 64, 64, 3, [2, 2, 2], 2, p_none=0.0)
    dev = harness.upload_dense(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    plan.T = 12                           # the caller lies about T
    mb.mint_lora_apply_fused(dev.pool, dev.table, plan, dev.x[:12], dev.y[:12], dev.status)
    torch.cuda.synchronize()
    assert dev.status[0].item() == mb.MINT_ERR_SHAPE_MISMATCH
    np.testing.assert_array_equal(mb.bits_from_bf16(dev.y), case.y0)


def test_host_side_argument_checks():
    from paper_2605_13779_b200 import binding as mb, harness
    case = synth.random_dense_case("gpu/args", 16, 64, 64, 3, [2, 2, 2], 2, p_none=0.0)
    dev = harness.upload_dense(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    with pytest.raises(mb.MintError) as e:      # misaligned activation pointer
        mb.mint_lora_apply_fused(dev.pool, dev.table, plan, dev.x.view(-1)[1:].view(-1)[: 15 * 64].view(15, 64),
                                 dev.y, dev.status)
    assert e.value.status == mb.MINT_ERR_MISALIGNED
    other = mb.SlotTable(10, 5)
    with pytest.raises(mb.MintError) as e:      # pool and table disagree on the slot count
        mb.mint_lora_apply_fused(dev.pool, other, plan, dev.x, dev.y, dev.status)
    assert e.value.status == mb.MINT_ERR_SHAPE_MISMATCH
    big = mb.SlotTable(10, 3)
    big.bind(0, 0, 64, 1.0)
    with pytest.raises(mb.MintError) as e:      # a bound adapter is wider than the pool's slots
        mb.mint_lora_apply_fused(dev.pool, big, plan, dev.x, dev.y, dev.status)
    assert e.value.status == mb.MINT_ERR_RANK_TOO_LARGE
    small = torch.empty(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(mb.MintError) as e:
        mb.load_library().mint_lora_plan  # noqa: B018
        p2 = mb.Plan(16, 1, 3, 0)
        p2.blob, p2.nbytes = small, 64
        mb.mint_lora_plan(dev.table, dev.ids, dev.status, plan=p2)
    assert e.value.status == mb.MINT_ERR_WORKSPACE_TOO_SMALL
    moe_pool = mb.Pool(dev.pool.A, dev.pool.B, 64, 64, 2, 3, num_experts=1)
    with pytest.raises(mb.MintError) as e:      # dense call on a packed MoE pool
        mb.mint_lora_apply_fused(moe_pool, dev.table, plan, dev.x, dev.y, dev.status)
    assert e.value.status == mb.MINT_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    np.testing.assert_array_equal(mb.bits_from_bf16(dev.y), case.y0)     # none of the refused calls ran


def test_slot_admission_writes_only_the_adapter_rows():
    """write_slot copies an adapter into its slot; the result equals a pool
    uploaded whole, and padding rows keep what they held."""
    from paper_2605_13779_b200 import binding as mb, harness
    case = synth.random_dense_case("gpu/admit", 24, 128, 64, 3, [2, 4, 1], 4, p_none=0.0)
    y_ref, _, _ = parity.oracle_dense(case)
    dev = harness.upload_dense(case)
    A = torch.full_like(dev.pool.A, float("nan"))
    B = torch.full_like(dev.pool.B, float("nan"))
    pool = mb.Pool(A, B, case.d, case.n, case.r_max, 3)
    for slot in range(3):
        r = int(case.table.slot_rank[slot])
        a_src = mb.bf16_from_bits(case.A[slot, :r], "cuda" if slot != 1 else "cpu")
        b_src = mb.bf16_from_bits(case.B[slot, :r], "cuda" if slot != 1 else "cpu")
        pool.write_slot(slot, a_src, b_src, r)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    mb.mint_lora_apply_fused(pool, dev.table, plan, dev.x, dev.y, dev.status)
    torch.cuda.synchronize()
    parity.assert_close(harness.y_to_f64(dev.y), y_ref, "admitted pool")
    assert torch.isnan(A[0, 2:]).all() and torch.isnan(B[2, 1:]).all()
    with pytest.raises(mb.MintError) as e:
        pool.write_slot(0, a_src, b_src, 9)
    assert e.value.status == mb.MINT_ERR_RANK_TOO_LARGE


def test_moe_slot_admission():
    from paper_2605_13779_b200 import binding as mb, harness
    batch = synth.config4_batch(T=12, E=3, K=2, num_slots=2, rank=3, tag="gpu/moeadmit")
    case = synth.config4_projection(batch, "gate", d=64, n=32, tag="gpu/moeadmit")
    # same adapters stored in wider (r_max = 8) slots through write_slot
    A = torch.full((2, 3, 64, 8), float("nan"), dtype=torch.bfloat16, device="cuda")
    B = torch.full((2, 3, 8, 32), float("nan"), dtype=torch.bfloat16, device="cuda")
    pool = mb.Pool(A, B, 64, 32, 8, 2, num_experts=3)
    for s in range(2):
        for e in range(3):
            pool.write_slot(s, mb.bf16_from_bits(case.A[s, e]), mb.bf16_from_bits(case.B[s, e]), 3, expert=e)
    dev = harness.upload_moe(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status, expert_ids=dev.expert_ids, num_experts=3)
    mb.mint_moe_lora_apply(pool, dev.table, plan, dev.x, dev.y, dev.status, x_row=dev.x_row)
    torch.cuda.synchronize()
    y_ref, _ = parity.oracle_moe(case)
    parity.assert_close(harness.y_to_f64(dev.y), y_ref, "moe admitted pool")


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """The tensor-core shrink of a batch with dense segments, with its tensor-core work withheld:
    nothing ever signals the barriers its CTAs wait on, so every wait runs out after its limit.
    The kernel reports MINT_ERR_TIMEOUT, writes nothing, frees its tensor memory and returns; the
    next ordinary call on the same stream is correct."""
    import time
    from paper_2605_13779_b200 import binding as mb, harness, synth
    import parity
    import test_gpu_dense as dense
    case = dense.dense_segment_case("gpu/timeout", [700, 130, 128, 3000, 300], [0, 1, 2, 3, 1], [64, 16, 8, 33],
                                    d=1032, n=520, r_max=64)
    assert case.T >= 4096
    dev = harness.upload_dense(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    ws = mb.new_workspace(dev.pool, case.T)
    ws.fill_(0x5A)
    before = ws.clone()
    y_before = dev.y.clone()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    mb.mint_selftest_wait_timeout(dev.pool, dev.table, plan, dev.x, dev.status, ws)
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    st = dev.status.cpu().numpy()
    assert st[0] == mb.MINT_ERR_TIMEOUT, st
    assert elapsed < 2.0                       # milliseconds per wait, not the second of the apply path
    assert torch.equal(ws, before)             # no part of v was written
    assert torch.equal(dev.y, y_before)
    # the context is intact: the ordinary apply right after it matches the oracle
    status = mb.new_status()
    mb.mint_lora_apply_fused(dev.pool, dev.table, plan, dev.x, dev.y, status, workspace=ws)
    torch.cuda.synchronize()
    assert status[0].item() == 0
    y_ref, _, _ = parity.oracle_dense(case)
    parity.assert_close(harness.y_to_f64(dev.y), y_ref, "apply after a timed-out wait")


def test_host_side_argument_checks_of_the_backward_and_the_grouped_moe_call():
    from paper_2605_13779_b200 import binding as mb, harness
    case = synth.random_dense_case("gpu/args-bwd", 16, 64, 64, 3, [2, 2, 2], 2, p_none=0.0)
    dev = harness.upload_dense(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    dy = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    dx = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    dA = torch.zeros(3, 2, 64, dtype=torch.float32, device="cuda")
    dB = torch.zeros(3, 2, 64, dtype=torch.float32, device="cuda")
    with pytest.raises(mb.MintError) as e:      # the weight gradients come together
        mb.mint_lora_backward(dev.pool, dev.table, plan, dev.x, dy, dev.status, dx=dx, dA=dA, dB=None)
    assert e.value.status == mb.MINT_ERR_INVALID_ARG
    with pytest.raises(mb.MintError) as e:      # a workspace that is too small
        mb.mint_lora_backward(dev.pool, dev.table, plan, dev.x, dy, dev.status, dx=dx, dA=dA, dB=dB,
                              workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == mb.MINT_ERR_WORKSPACE_TOO_SMALL
    moe_pool = mb.Pool(dev.pool.A, dev.pool.B, 64, 64, 2, 3, num_experts=1)
    with pytest.raises(mb.MintError) as e:      # the backward takes rank-major pools only
        mb.mint_lora_backward(moe_pool, dev.table, plan, dev.x, dy, dev.status, dx=dx, dA=dA, dB=dB)
    assert e.value.status == mb.MINT_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert float(dA.abs().sum()) == 0.0 and float(dx.float().abs().sum()) == 0.0   # none of the refused calls ran

    # grouped MoE call: pools with different expert counts, a dense pool among the items
    batch = synth.config4_batch(T=8, E=4, K=2, num_slots=2, rank=8, tag="gpu/args-moe")
    mcase = synth.config4_projection(batch, "gate", d=64, n=64, tag="gpu/args-moe")
    mdev = harness.upload_moe(mcase)
    mplan = mb.mint_lora_plan(mdev.table, mdev.ids, mdev.status, expert_ids=mdev.expert_ids, num_experts=4)
    ws = mb.new_moe_workspace(mdev.pool, 8, 2)
    fewer = mb.Pool(mdev.pool.A, mdev.pool.B, 64, 64, 8, 2, num_experts=2)
    with pytest.raises(mb.MintError) as e:
        mb.mint_moe_lora_apply_grouped([(mdev.pool, mdev.x, mdev.y, ws), (fewer, mdev.x, mdev.y, ws)], mdev.table,
                                       mplan, mdev.status, x_row=mdev.x_row)
    assert e.value.status == mb.MINT_ERR_SHAPE_MISMATCH
    dense_pool = mb.Pool(mdev.pool.A, mdev.pool.B, 64, 64, 8, 2)
    with pytest.raises(mb.MintError) as e:
        mb.mint_moe_lora_apply_grouped([(dense_pool, mdev.x, mdev.y, ws)], mdev.table, mplan, mdev.status,
                                       x_row=mdev.x_row)
    assert e.value.status == mb.MINT_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    np.testing.assert_array_equal(mb.bits_from_bf16(mdev.y), mcase.y0)

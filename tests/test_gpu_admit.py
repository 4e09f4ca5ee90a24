"""Admission from the packed representation and the slot manager on the GPU:
pool bytes against the CPU scatter of oracle/admission.py, and
admit-then-apply against the apply oracle."""
import numpy as np
import pytest
import torch

from oracle import admission
from paper_2605_13779_b200 import synth
import parity

pytestmark = pytest.mark.gpu


def bits(t):
    from paper_2605_13779_b200 import binding as mb
    return mb.bits_from_bf16(t)


@pytest.mark.parametrize("E,d,n,r_max,rank", [
    (4, 72, 40, 16, 16), (4, 72, 40, 16, 1), (3, 64, 8, 16, 3), (8, 264, 136, 32, 8), (2, 16, 16, 8, 8),
    (5, 40, 24, 1, 1), (128, 2048, 768, 16, 1),
])
def test_packed_moe_admission_writes_exactly_the_slot(E, d, n, r_max, rank):
    from paper_2605_13779_b200 import binding as mb
    rng = synth.stream("gpu/admit", E, d, n, r_max, rank)
    S, slot = 3, 1
    A0 = np.full((S, E, d, r_max), synth.BF16_NAN_BITS, dtype=np.uint16)
    B0 = np.full((S, E, r_max, n), synth.BF16_NAN_BITS, dtype=np.uint16)
    A_src = synth.normal_bf16(rng, (E, d, rank), 0.02)
    B_src = synth.normal_bf16(rng, (E, rank, n), 0.02)
    A, B = mb.bf16_from_bits(A0), mb.bf16_from_bits(B0)
    pool = mb.Pool(A, B, d, n, r_max, S, num_experts=E)
    pool.admit_packed(slot, mb.bf16_from_bits(A_src), mb.bf16_from_bits(B_src), rank)
    torch.cuda.synchronize()
    admission.admit_packed_moe(A0, B0, slot, A_src, B_src, rank)
    np.testing.assert_array_equal(bits(A), A0)
    np.testing.assert_array_equal(bits(B), B0)


@pytest.mark.parametrize("d,n,r_max,rank", [(2560, 1024, 32, 32), (264, 72, 12, 5), (64, 64, 1, 1)])
def test_dense_admission_writes_exactly_the_slot(d, n, r_max, rank):
    from paper_2605_13779_b200 import binding as mb
    rng = synth.stream("gpu/admit/dense", d, n, r_max, rank)
    S, slot = 4, 2
    A0 = np.full((S, r_max, d), synth.BF16_NAN_BITS, dtype=np.uint16)
    B0 = np.full((S, r_max, n), synth.BF16_NAN_BITS, dtype=np.uint16)
    A_src = synth.normal_bf16(rng, (rank, d), 0.02)
    B_src = synth.normal_bf16(rng, (rank, n), 0.02)
    A, B = mb.bf16_from_bits(A0), mb.bf16_from_bits(B0)
    pool = mb.Pool(A, B, d, n, r_max, S)
    pool.admit_packed(slot, mb.bf16_from_bits(A_src), mb.bf16_from_bits(B_src), rank)
    torch.cuda.synchronize()
    admission.admit_packed_dense(A0, B0, slot, A_src, B_src, rank)
    np.testing.assert_array_equal(bits(A), A0)
    np.testing.assert_array_equal(bits(B), B0)


def test_admission_rejects_bad_arguments():
    from paper_2605_13779_b200 import binding as mb
    A = torch.zeros(2, 2, 16, 8, dtype=torch.bfloat16, device="cuda")
    B = torch.zeros(2, 2, 8, 16, dtype=torch.bfloat16, device="cuda")
    pool = mb.Pool(A, B, 16, 16, 8, 2, num_experts=2)
    src_a = torch.zeros(2, 16, 8, dtype=torch.bfloat16, device="cuda")
    src_b = torch.zeros(2, 8, 16, dtype=torch.bfloat16, device="cuda")
    for slot, rank, code in ((2, 8, mb.MINT_ERR_INVALID_ARG), (0, 9, mb.MINT_ERR_RANK_TOO_LARGE),
                             (0, 0, mb.MINT_ERR_INVALID_ARG)):
        with pytest.raises(mb.MintError) as e:
            pool.admit_packed(slot, src_a, src_b, rank)
        assert e.value.status == code


def test_admit_then_apply_equals_apply_on_a_pool_uploaded_whole():
    """A 30B-A3B-shaped MoE projection at reduced size: every slot admitted from its
    packed tensors (mixed ranks) gives the same pool bytes as the whole upload, and
    the apply over it matches the oracle."""
    import dataclasses
    from paper_2605_13779_b200 import binding as mb, harness
    tag = "gpu/admit/apply"
    ranks = [16, 1, 8, 3]
    batch = synth.config4_batch(T=96, E=8, K=2, num_slots=4, rank=16, tag=tag)
    batch = dataclasses.replace(batch, table=synth.identity_table(4, np.asarray(ranks, dtype=np.int32), 2.0))
    case = synth.config4_projection(batch, "gate", d=520, n=264, tag=tag)
    whole = harness.upload_moe(case)
    A = torch.full_like(whole.pool.A, float("nan"))
    B = torch.full_like(whole.pool.B, float("nan"))
    pool = mb.Pool(A, B, case.d, case.n, case.r_max, 4, num_experts=case.E)
    for s, r in enumerate(ranks):
        A_src = mb.bf16_from_bits(np.ascontiguousarray(case.A[s, :, :, :r]))
        B_src = mb.bf16_from_bits(np.ascontiguousarray(case.B[s, :, :r, :]))
        pool.admit_packed(s, A_src, B_src, r)
    torch.cuda.synchronize()
    # same bytes wherever the whole upload holds weights (its padding is NaN too)
    np.testing.assert_array_equal(bits(A), case.A)
    np.testing.assert_array_equal(bits(B), case.B)
    plan = mb.mint_lora_plan(whole.table, whole.ids, whole.status, expert_ids=whole.expert_ids, num_experts=case.E)
    mb.mint_moe_lora_apply(pool, whole.table, plan, whole.x, whole.y, whole.status, x_row=whole.x_row)
    torch.cuda.synchronize()
    assert whole.status[0].item() == 0
    y_ref, _ = parity.oracle_moe(case)
    parity.assert_close(harness.y_to_f64(whole.y), y_ref, "admit then apply")


def test_slot_manager_with_a_table_evicts_binds_and_invalidates_plans():
    """Three slots, four adapters: the fourth takes the slot of the least recently used one;
    tokens naming the evicted adapter are reported as not resident; a plan made before the
    change is refused as stale; the apply over the new residents matches the oracle."""
    from paper_2605_13779_b200 import binding as mb, harness
    d, n, r_max, S = 256, 128, 8, 3
    ranks = {100: 8, 200: 4, 300: 1, 400: 8}
    rng = synth.stream("gpu/admit/manager")
    weights = {cid: (synth.normal_bf16(rng, (r, d), 0.02), synth.normal_bf16(rng, (r, n), 0.02))
               for cid, r in ranks.items()}
    table = mb.SlotTable(1000, S)
    mgr = mb.SlotManager(S, table)
    A = torch.full((S, r_max, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    B = torch.full((S, r_max, n), float("nan"), dtype=torch.bfloat16, device="cuda")
    pool = mb.Pool(A, B, d, n, r_max, S)
    model = admission.LruSlots(S)

    def acquire(cid):
        slot, admitted, evicted = mgr.acquire(cid, ranks[cid], 2.0)
        assert (slot, admitted, evicted) == model.acquire(cid)
        if admitted:
            pool.admit_packed(slot, mb.bf16_from_bits(weights[cid][0]), mb.bf16_from_bits(weights[cid][1]), ranks[cid])
        return slot

    for cid in (100, 200, 300):
        acquire(cid)
    for cid in (100, 200, 300):
        mgr.release(cid)
        model.release(cid)
    T = 40
    ids_np = rng.choice(np.array([100, 200, 300, 400, -1]), size=T).astype(np.int64)
    ids = torch.from_numpy(ids_np).cuda()
    x_bits = synth.normal_bf16(rng, (T, d), 1.0)
    y_bits = synth.normal_bf16(rng, (T, n), 1.0)
    status = mb.new_status()
    old_plan = mb.mint_lora_plan(table, ids, status)
    torch.cuda.synchronize()
    assert status[0].item() == mb.MINT_ERR_NOT_RESIDENT and status[1].item() == int((ids_np == 400).sum())

    gen = table.generation
    acquire(200)                 # touch: 100 is now the least recently used
    slot400 = acquire(400)
    assert slot400 == 0 and mgr.lookup(100) == -1 and table.generation > gen
    x, y = mb.bf16_from_bits(x_bits), mb.bf16_from_bits(y_bits)
    status = mb.new_status()
    mb.mint_lora_apply_fused(pool, table, old_plan, x, y, status)     # made under the old bindings
    torch.cuda.synchronize()
    assert status[0].item() == mb.MINT_ERR_STALE_PLAN
    np.testing.assert_array_equal(bits(y), y_bits)

    status = mb.new_status()
    plan = mb.mint_lora_plan(table, ids, status)
    mb.mint_lora_apply_fused(pool, table, plan, x, y, status)
    torch.cuda.synchronize()
    assert status[0].item() == mb.MINT_ERR_NOT_RESIDENT and status[1].item() == int((ids_np == 100).sum())
    # oracle over the same residency
    id_to_slot = np.full(1000, -1, dtype=np.int32)
    slot_rank = np.zeros(S, dtype=np.int32)
    A_ref = np.full((S, r_max, d), synth.BF16_NAN_BITS, dtype=np.uint16)
    B_ref = np.full((S, r_max, n), synth.BF16_NAN_BITS, dtype=np.uint16)
    for cid, slot in model.resident().items():
        id_to_slot[cid] = slot
        slot_rank[slot] = ranks[cid]
        admission.admit_packed_dense(A_ref, B_ref, slot, weights[cid][0], weights[cid][1], ranks[cid])
    from oracle import oracle
    y_ref, _, missing = oracle.lora_apply(ids_np, id_to_slot, slot_rank, np.full(S, 2.0, dtype=np.float32), A_ref, B_ref,
                                          x_bits, y_bits)
    assert missing == int((ids_np == 100).sum())
    parity.assert_close(harness.y_to_f64(y), y_ref, "apply after eviction")
    gone = (ids_np == 100) | (ids_np == -1)
    np.testing.assert_array_equal(bits(y)[gone], y_bits[gone])

"""Pins for the fp64 CPU oracle of the LoRA apply (CPU only).

Each test ties the oracle to something other than itself: hand-computed
examples, identities of the definition y = y0 + s (x A) B, special cases that
reduce to a numpy matrix product, and brute-force merged weights W + s A B."""
import numpy as np
import pytest

from oracle import oracle
from paper_2605_13779_b200 import synth
from golden_io import read_golden


def bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def f64(b):
    return synth.bf16_bits_to_f64(b)


def run_case(case, **kw):
    t = case.table
    return oracle.lora_apply(case.ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                             case.A, case.B, case.x, case.y0, **kw)


def small_case(name="pin", T=24, d=48, n=40, num_slots=5, ranks=(1, 2, 3, 4, 4), r_max=4, **kw):
    return synth.random_dense_case(name, T, d, n, num_slots, list(ranks), r_max, **kw)


def test_golden_dense_example():
    g = read_golden("dense_tiny.txt")
    d, n, r_max = int(g["d"][0]), int(g["n"][0]), int(g["r_max"][0])
    A = np.full((2, r_max, d), np.nan, dtype=np.float32)   # [slot][rank row][d]; padding = NaN
    B = np.full((2, r_max, n), np.nan, dtype=np.float32)
    A0 = np.atleast_2d(g["A0"]); A1 = np.atleast_2d(g["A1"]).reshape(d, 1)
    A[0, :2, :] = A0.T
    A[1, :1, :] = A1.T
    B[0, :2, :] = g["B0"]
    B[1, :1, :] = np.atleast_2d(g["B1"])
    y, v, missing = oracle.lora_apply(
        g["ids"].astype(np.int64), np.array([0, 1], np.int32), g["rank"].astype(np.int32),
        g["scale"].astype(np.float32), bits(A), bits(B), bits(g["x"]), bits(g["y0"]), want_v=True)
    assert missing == 0
    np.testing.assert_array_equal(y, g["y"])
    np.testing.assert_array_equal(v, g["v"])


def test_golden_dense_example_dr_layout():
    """Same example with A stored [slot][d][r]: the stride arguments, not the
    storage order, define the operand."""
    g = read_golden("dense_tiny.txt")
    A = np.full((2, 2, 2), np.nan, dtype=np.float32)        # [slot][d][r_max]
    A[0] = g["A0"]
    A[1, :, 0] = g["A1"].reshape(-1)
    B = np.full((2, 2, 3), np.nan, dtype=np.float32)
    B[0] = g["B0"]
    B[1, 0] = g["B1"]
    y, _, _ = oracle.lora_apply(
        g["ids"].astype(np.int64), np.array([0, 1], np.int32), g["rank"].astype(np.int32),
        g["scale"].astype(np.float32), bits(A), bits(B), bits(g["x"]), bits(g["y0"]), a_layout="dr")
    np.testing.assert_array_equal(y, g["y"])


def test_no_adapter_and_zero_B_leave_y_unchanged():
    case = small_case("pin/none", p_none=0.4)
    assert (case.ids == -1).any() and (case.ids >= 0).any()
    y, _, missing = run_case(case)
    none = case.ids == -1
    np.testing.assert_array_equal(y[none], f64(case.y0)[none])
    assert np.abs(y[~none] - f64(case.y0)[~none]).max() > 0
    # B = 0 for every adapter (padding stays NaN: it must not be read)
    B0 = case.B.copy()
    B0[B0 != synth.BF16_NAN_BITS] = 0
    t = case.table
    y2, _, _ = oracle.lora_apply(case.ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                 case.A, B0, case.x, case.y0)
    np.testing.assert_array_equal(y2, f64(case.y0))
    assert missing == 0


def test_padding_rows_are_never_read():
    case = small_case("pin/pad", p_none=0.0)
    y, _, _ = run_case(case)
    assert np.isfinite(y).all()
    A2, B2 = case.A.copy(), case.B.copy()
    A2[A2 == synth.BF16_NAN_BITS] = bits(np.float32(123.0))
    B2[B2 == synth.BF16_NAN_BITS] = bits(np.float32(-77.0))
    t = case.table
    y2, _, _ = oracle.lora_apply(case.ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                 A2, B2, case.x, case.y0)
    np.testing.assert_array_equal(y, y2)


def test_rank1_is_outer_product_update():
    case = small_case("pin/rank1", T=16, d=64, n=32, num_slots=3, ranks=(1, 1, 1), r_max=1, p_none=0.0)
    y, v, _ = run_case(case, want_v=True)
    x, y0 = f64(case.x), f64(case.y0)
    for t in range(case.T):
        a = f64(case.A[case.ids[t], 0])          # d-vector
        b = f64(case.B[case.ids[t], 0])          # n-vector
        dot = float(np.dot(x[t], a))
        np.testing.assert_allclose(v[t, 0], dot, rtol=1e-13, atol=1e-15)
        np.testing.assert_allclose(y[t], y0[t] + 2.0 * dot * b, rtol=1e-13, atol=1e-15)


def test_linear_in_scale():
    case = small_case("pin/lin", p_none=0.1)
    t = case.table
    y0 = f64(case.y0)
    ya, _, _ = run_case(case)
    s2 = (t.slot_scale * np.float32(-3.5)).astype(np.float32)
    yb, _, _ = oracle.lora_apply(case.ids, t.id_to_slot, t.slot_rank, s2, case.A, case.B, case.x, case.y0)
    np.testing.assert_allclose(yb - y0, -3.5 * (ya - y0), rtol=1e-12, atol=1e-14)


def test_token_permutation_equivariance():
    case = small_case("pin/perm", p_none=0.2)
    t = case.table
    y, _, _ = run_case(case)
    p = synth.stream("pin/perm/p").permutation(case.T)
    yp, _, _ = oracle.lora_apply(case.ids[p], t.id_to_slot, t.slot_rank, t.slot_scale,
                                 case.A, case.B, case.x[p], case.y0[p])
    np.testing.assert_array_equal(yp, y[p])


def test_single_adapter_equals_two_matmuls():
    """One adapter for all tokens: y = y0 + s (X A) B, two library matrix products."""
    case = small_case("pin/mm", T=33, d=96, n=72, num_slots=2, ranks=(4, 3), r_max=4, p_none=0.0)
    for slot in (0, 1):
        ids = np.full(case.T, slot, dtype=np.int64)
        t = case.table
        y, _, _ = oracle.lora_apply(ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                    case.A, case.B, case.x, case.y0)
        r = int(t.slot_rank[slot])
        Amat = f64(case.A[slot, :r]).T            # d x r
        Bmat = f64(case.B[slot, :r])              # r x n
        expect = f64(case.y0) + 2.0 * (f64(case.x) @ Amat) @ Bmat
        np.testing.assert_allclose(y, expect, rtol=1e-12, atol=1e-13)


def test_tiny_matches_merged_weights():
    """y0 = x W; the apply must give x (W + s A B): the merged-checkpoint path
    the paper contrasts the adapter path with (handoff figure, Introduction)."""
    rng = synth.stream("pin/merged")
    T, d, n, r = 8, 16, 12, 4
    # small integers keep x W exact in bf16-free fp64 and representable inputs in bf16
    x = rng.integers(-3, 4, size=(T, d)).astype(np.float64)
    W = rng.integers(-2, 3, size=(d, n)).astype(np.float64)
    num_slots = 3
    Amat = rng.integers(-2, 3, size=(num_slots, d, r)).astype(np.float64)
    Bmat = rng.integers(-2, 3, size=(num_slots, r, n)).astype(np.float64)
    scale = np.array([2.0, 0.5, -1.0], dtype=np.float32)
    rank = np.array([4, 2, 3], dtype=np.int32)
    ids = rng.integers(0, num_slots, size=T).astype(np.int64)
    y0 = x @ W
    assert np.abs(y0).max() < 256          # exact in bf16
    A_store = np.full((num_slots, r, d), np.nan, dtype=np.float32)
    B_store = np.full((num_slots, r, n), np.nan, dtype=np.float32)
    for s in range(num_slots):
        A_store[s, :rank[s]] = Amat[s, :, :rank[s]].T
        B_store[s, :rank[s]] = Bmat[s, :rank[s]]
    y, _, _ = oracle.lora_apply(ids, np.arange(num_slots, dtype=np.int32), rank, scale,
                                bits(A_store), bits(B_store), bits(x), bits(y0))
    for t in range(T):
        s = ids[t]
        Wm = W + float(scale[s]) * Amat[s, :, :rank[s]] @ Bmat[s, :rank[s]]
        np.testing.assert_allclose(y[t], x[t] @ Wm, rtol=1e-12, atol=1e-12)


def test_mixed_batch_rows_equal_isolated_adapter_rows():
    case = small_case("pin/iso", T=40, p_none=0.1)
    t = case.table
    y, _, _ = run_case(case)
    for a in range(t.num_slots):
        sel = np.nonzero(case.ids == a)[0]
        if sel.size == 0:
            continue
        ya, _, _ = oracle.lora_apply(case.ids[sel], t.id_to_slot, t.slot_rank, t.slot_scale,
                                     case.A, case.B, case.x[sel], case.y0[sel])
        np.testing.assert_array_equal(ya, y[sel])


def test_non_resident_ids_are_counted_and_left_untouched():
    case = small_case("pin/missing", p_none=0.0)
    t = case.table
    table = t.id_to_slot.copy()
    table[2] = -1
    ids = case.ids.copy()
    ids[0] = 2
    ids[1] = 10_000      # outside the catalog
    y, _, missing = oracle.lora_apply(ids, table, t.slot_rank, t.slot_scale, case.A, case.B, case.x, case.y0)
    gone = (ids == 2) | (ids == 10_000)
    assert missing == int(gone.sum())
    np.testing.assert_array_equal(y[gone], f64(case.y0)[gone])


def test_slot_table_indirection():
    """Catalog id -> slot through a non-identity table equals the identity
    table with ids rewritten to slots."""
    case = small_case("pin/table", p_none=0.1)
    t = case.table
    rng = synth.stream("pin/table/cat")
    catalog = 1000
    cat_ids = rng.choice(catalog, size=t.num_slots, replace=False)
    table = np.full(catalog, -1, dtype=np.int32)
    table[cat_ids] = np.arange(t.num_slots, dtype=np.int32)
    ids2 = np.where(case.ids >= 0, cat_ids[np.maximum(case.ids, 0)], -1)
    y1, _, _ = run_case(case)
    y2, _, m = oracle.lora_apply(ids2, table, t.slot_rank, t.slot_scale, case.A, case.B, case.x, case.y0)
    assert m == 0
    np.testing.assert_array_equal(y1, y2)


# ---------------------------------------------------------------- MoE ------
def moe_small(name="pin/moe", T=12, K=2, E=4, d=32, n=24, num_slots=3, rank=3, p_none=0.1):
    batch = synth.config4_batch(T=T, E=E, K=K, num_slots=num_slots, rank=rank, p_none=p_none, tag=name)
    return synth.config4_projection(batch, "gate", d=d, n=n, tag=name)


def run_moe(case, **kw):
    t = case.table
    kw.setdefault("x_row", case.x_row)
    return oracle.moe_lora_apply(case.ids, case.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                 case.A, case.B, case.x, case.y0, **kw)


def test_golden_moe_example():
    g = read_golden("moe_tiny.txt")
    A = np.zeros((1, 2, 2, 1), dtype=np.float32)      # [slot][E][d][r]
    A[0, 0, :, 0] = g["A_e0"].reshape(-1)
    A[0, 1, :, 0] = g["A_e1"].reshape(-1)
    B = np.zeros((1, 2, 1, 2), dtype=np.float32)      # [slot][E][r][n]
    B[0, 0, 0] = g["B_e0"]
    B[0, 1, 0] = g["B_e1"]
    args = (g["ids"].astype(np.int64), g["experts"].astype(np.int32).reshape(1, 2),
            np.array([0], np.int32), np.array([1], np.int32), np.array([1.0], np.float32),
            bits(A), bits(B), bits(np.atleast_2d(g["x"])), bits(g["y0"]))
    xr = g["x_row"].astype(np.int32)
    y, _ = oracle.moe_lora_apply(*args, x_row=xr)
    np.testing.assert_array_equal(y, g["y_unweighted"])
    yw, _ = oracle.moe_lora_apply(*args, x_row=xr, pair_weight=g["weights"].astype(np.float32))
    np.testing.assert_array_equal(yw, g["y_weighted"])


def test_moe_one_expert_top1_reduces_to_dense():
    case = moe_small("pin/moe1", T=10, K=1, E=1)
    y_moe, _ = run_moe(case)
    t = case.table
    A_dense = case.A[:, 0]                             # [slot][d][r]
    B_dense = case.B[:, 0]
    y_dense, _, _ = oracle.lora_apply(case.ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                      A_dense, B_dense, case.x, case.y0, a_layout="dr")
    np.testing.assert_array_equal(y_moe, y_dense)


def test_moe_group_equals_matmul():
    """All pairs of one (expert, slot) group: Y = Y0 + s (X A[slot][e]) B[slot][e]."""
    case = moe_small("pin/moemm", T=40, p_none=0.0)
    y, _ = run_moe(case)
    P = case.T * case.K
    pair_slot = np.repeat(case.ids, case.K)
    pair_exp = case.expert_ids.reshape(-1)
    checked = 0
    for e in range(case.E):
        for s in range(case.table.num_slots):
            sel = np.nonzero((pair_exp == e) & (pair_slot == s))[0]
            if sel.size == 0:
                continue
            X = f64(case.x)[case.x_row[sel]]
            Am = f64(case.A[s, e])[:, :case.table.slot_rank[s]]
            Bm = f64(case.B[s, e])[:case.table.slot_rank[s]]
            expect = f64(case.y0)[sel] + 2.0 * (X @ Am) @ Bm
            np.testing.assert_allclose(y[sel], expect, rtol=1e-12, atol=1e-13)
            checked += sel.size
    assert checked == P


def test_moe_constant_pair_weight_scales_delta():
    case = moe_small("pin/moew")
    y1, _ = run_moe(case)
    w = np.full(case.T * case.K, 0.375, dtype=np.float32)
    yw, _ = run_moe(case, pair_weight=w)
    y0 = f64(case.y0)
    np.testing.assert_allclose(yw - y0, 0.375 * (y1 - y0), rtol=1e-12, atol=1e-14)


def test_moe_expert_relabel_invariance():
    case = moe_small("pin/moeperm")
    y1, _ = run_moe(case)
    q = synth.stream("pin/moeperm/q").permutation(case.E)      # new label of expert e is q[e]
    A2 = np.empty_like(case.A); B2 = np.empty_like(case.B)
    A2[:, q] = case.A
    B2[:, q] = case.B
    t = case.table
    y2, _ = oracle.moe_lora_apply(case.ids, q[case.expert_ids].astype(np.int32), t.id_to_slot, t.slot_rank,
                                  t.slot_scale, A2, B2, case.x, case.y0, x_row=case.x_row)
    np.testing.assert_array_equal(y1, y2)


def test_moe_down_projection_reads_pair_rows():
    batch = synth.config4_batch(T=6, E=4, K=2, num_slots=2, rank=2, tag="pin/moedown")
    case = synth.config4_projection(batch, "down", d=16, n=8, tag="pin/moedown")
    assert case.x_row is None and case.x.shape[0] == 12
    y, _ = run_moe(case)
    ident = np.arange(12, dtype=np.int32)
    y2, _ = run_moe(case, x_row=ident)
    np.testing.assert_array_equal(y, y2)


# ------------------------------------------------------- tolerance budget --
def test_bf16_store_error_budget():
    """Rounding an N(0,1)-like output to bf16 (8 significant bits: relative
    half-ulp between 2^-9 and 2^-8) costs about 1.7e-3 relative Frobenius
    error: the stated 5e-3 bound leaves room for it, and 3e-2 exceeds the
    half-ulp (2^-6) of every |y| < 8."""
    rng = synth.stream("pin/budget")
    y = rng.standard_normal(1 << 18)
    yr = synth.bf16_bits_to_f64(synth.f32_to_bf16_bits(y.astype(np.float32)))
    rel = np.linalg.norm(yr - y) / np.linalg.norm(y)
    assert 2.0 ** -9 / np.sqrt(3) < rel < 2.0 ** -8 / np.sqrt(3)
    assert np.abs(yr - y).max() <= 2.0 ** -6 + 1e-12        # half-ulp for |y| in [4, 8)


def test_combine_oracle_equals_explicit_weighted_sum_on_a_tiny_case():
    """Brute force: Y[t] = Y0[t] + sum_k w s x A B with every product written out in numpy."""
    from paper_2605_13779_b200 import synth
    batch = synth.config4_batch(T=5, E=3, K=2, num_slots=2, rank=2, tag="oracle/combine")
    case = synth.config4_projection(batch, "down", d=8, n=6, tag="oracle/combine")
    y0 = synth.normal_bf16(synth.stream("oracle/combine/y0"), (case.T, case.n), 1.0)
    t = case.table
    got, missing = oracle.moe_lora_apply_combine(case.ids, case.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                                 case.A, case.B, case.x, y0, case.pair_weight)
    assert missing == 0
    A = synth.bf16_bits_to_f64(case.A)
    B = synth.bf16_bits_to_f64(case.B)
    x = synth.bf16_bits_to_f64(case.x)
    want = synth.bf16_bits_to_f64(y0).copy()
    for tok in range(case.T):
        s = t.id_to_slot[case.ids[tok]]
        for k in range(case.K):
            p = tok * case.K + k
            e = case.expert_ids[tok, k]
            r = t.slot_rank[s]
            v = x[p] @ A[s, e][:, :r]
            want[tok] += float(case.pair_weight[p]) * float(t.slot_scale[s]) * (v @ B[s, e][:r, :])
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-14)


def test_combine_oracle_with_one_expert_per_token_is_the_per_pair_apply():
    from paper_2605_13779_b200 import synth
    batch = synth.config4_batch(T=9, E=4, K=1, num_slots=3, rank=4, tag="oracle/combine1")
    case = synth.config4_projection(batch, "down", d=16, n=8, tag="oracle/combine1")
    t = case.table
    a, _ = oracle.moe_lora_apply_combine(case.ids, case.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                         case.A, case.B, case.x, case.y0, case.pair_weight)
    b, _ = oracle.moe_lora_apply(case.ids, case.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                 case.A, case.B, case.x, case.y0, pair_weight=case.pair_weight)
    np.testing.assert_allclose(a, b, rtol=1e-13, atol=1e-15)

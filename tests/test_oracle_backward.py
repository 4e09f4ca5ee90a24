"""Pins for the fp64 CPU oracle of the LoRA backward (CPU only).

The backward oracle is tied to things other than itself: a hand-computed example,
central differences of the FORWARD oracle (an independent C program), the closed
form for one adapter as numpy matrix products, and the masks (padding rows, empty
slots, tokens without an adapter)."""
import numpy as np
import pytest

from oracle import backward, oracle
from paper_2605_13779_b200 import synth
from golden_io import read_golden


def bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def f64(b):
    return synth.bf16_bits_to_f64(b)


def small_case(name="bwd-pin", T=20, d=24, n=16, num_slots=4, ranks=(1, 2, 3, 4), r_max=4, **kw):
    return synth.random_dense_case(name, T, d, n, num_slots, list(ranks), r_max, **kw)


def run_backward(case, dy, **kw):
    t = case.table
    return backward.lora_backward(case.ids, t.id_to_slot, t.slot_rank, t.slot_scale, case.A, case.B, case.x, dy, **kw)


def upstream(case, name="dy"):
    return synth.normal_bf16(synth.stream(case.name, name), (case.T, case.n), 1.0)


def test_golden_backward_example():
    g = read_golden("backward_tiny.txt")
    d, n, r_max = int(g["d"][0]), int(g["n"][0]), int(g["r_max"][0])
    A = np.full((2, r_max, d), np.nan, dtype=np.float32)   # padding = NaN: it must never be read
    B = np.full((2, r_max, n), np.nan, dtype=np.float32)
    A[0] = g["A0"]
    A[1, 0] = g["A1"]
    B[0] = g["B0"]
    B[1, 0] = g["B1"]
    dA0 = np.full((2, r_max, d), 7.0)                       # starting values show what is left alone
    dB0 = np.full((2, r_max, n), -3.0)
    dx, dA, dB, missing = backward.lora_backward(
        g["ids"].astype(np.int64), np.array([0, 1], np.int32), g["rank"].astype(np.int32),
        g["scale"].astype(np.float32), bits(A), bits(B), bits(g["x"]), bits(g["dy"]), dA0=dA0, dB0=dB0)
    assert missing == 0
    np.testing.assert_array_equal(dx, g["dx"])
    np.testing.assert_array_equal(dA[0], 7.0 + g["dA0"])
    np.testing.assert_array_equal(dB[0], -3.0 + g["dB0"])
    np.testing.assert_array_equal(dA[1, 0], 7.0 + g["dA1"])
    np.testing.assert_array_equal(dB[1, 0], -3.0 + g["dB1"])
    np.testing.assert_array_equal(dA[1, 1], np.full(d, 7.0))      # the padding row of slot 1
    np.testing.assert_array_equal(dB[1, 1], np.full(n, -3.0))


def forward_loss(case, dy, A=None, B=None, x=None):
    """L = sum(y * dy) with the forward oracle (its C implementation), y0 = 0."""
    t = case.table
    y, _, _ = oracle.lora_apply(case.ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                case.A if A is None else A, case.B if B is None else B,
                                case.x if x is None else x, np.zeros_like(case.y0))
    return float((y * f64(dy)).sum())


def test_central_differences_of_the_forward_oracle():
    """dL/dx, dL/dA, dL/dB by central differences of L = <y, dy> through the forward oracle.
    L is bilinear in (A, B) and linear in x, so a central difference with a power-of-two step
    is exact up to fp64 rounding; the step keeps the perturbed values exact in bf16."""
    case = small_case(p_none=0.15)
    dy = upstream(case)
    dx, dA, dB, _ = run_backward(case, dy)
    rng = np.random.default_rng(5)
    h = 0.5   # values are N(0,1) or N(0,0.02) in bf16: +-0.5 is exact for |v| < 4 only if the bits allow it,
              # so the probe REPLACES the value by (h, -h) around 0 and uses linearity: L(h) - L(-h) = 2 h dL/dv
    t = case.table
    for _ in range(12):   # x
        tt, c = int(rng.integers(case.T)), int(rng.integers(case.d))
        xp, xm = case.x.copy(), case.x.copy()
        xp[tt, c], xm[tt, c] = bits(h).item(), bits(-h).item()
        fd = (forward_loss(case, dy, x=xp) - forward_loss(case, dy, x=xm)) / (2 * h)
        assert fd == pytest.approx(dx[tt, c], rel=1e-9, abs=1e-9)
    used = np.unique(t.id_to_slot[case.ids[case.ids >= 0]])
    for _ in range(12):   # A and B, rows below the slot's rank of slots that have tokens
        slot = int(rng.choice(used))
        k = int(rng.integers(t.slot_rank[slot]))
        c = int(rng.integers(case.d))
        Ap, Am = case.A.copy(), case.A.copy()
        Ap[slot, k, c], Am[slot, k, c] = bits(h).item(), bits(-h).item()
        fd = (forward_loss(case, dy, A=Ap) - forward_loss(case, dy, A=Am)) / (2 * h)
        assert fd == pytest.approx(dA[slot, k, c], rel=1e-9, abs=1e-9)
        j = int(rng.integers(case.n))
        Bp, Bm = case.B.copy(), case.B.copy()
        Bp[slot, k, j], Bm[slot, k, j] = bits(h).item(), bits(-h).item()
        fd = (forward_loss(case, dy, B=Bp) - forward_loss(case, dy, B=Bm)) / (2 * h)
        assert fd == pytest.approx(dB[slot, k, j], rel=1e-9, abs=1e-9)


def test_one_adapter_is_three_matrix_products():
    """All tokens on one full-rank adapter: dx = s dy B^T A, dA = s (dy B^T)^T x, dB = s (x A^T)^T dy."""
    case = small_case(name="bwd-one", T=17, d=12, n=9, num_slots=1, ranks=(3,), r_max=3, p_none=0.0)
    dy = upstream(case)
    dx, dA, dB, _ = run_backward(case, dy)
    a, b, x, g = f64(case.A[0]), f64(case.B[0]), f64(case.x), f64(dy)
    s = float(case.table.slot_scale[0])
    np.testing.assert_allclose(dx, s * (g @ b.T) @ a, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dA[0], s * (g @ b.T).T @ x, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dB[0], s * (x @ a.T).T @ g, rtol=1e-12, atol=1e-12)


def test_masks_padding_rows_empty_slots_and_tokens_without_adapter():
    case = small_case(name="bwd-mask", T=12, num_slots=5, ranks=(1, 2, 3, 4, 2), p_none=0.3)
    ids = case.ids.copy()
    t = case.table
    ids[t.id_to_slot[np.maximum(ids, 0)] == 4] = -1    # slot 4 gets no token
    dy = upstream(case)
    dx0 = synth.normal_bf16(synth.stream(case.name, "dx0"), (case.T, case.d), 1.0)
    dA0 = np.full(case.A.shape, 2.5)
    dB0 = np.full(case.B.shape, -1.5)
    dx, dA, dB, missing = backward.lora_backward(ids, t.id_to_slot, t.slot_rank, t.slot_scale, case.A, case.B,
                                                 case.x, dy, dx0=dx0, dA0=dA0, dB0=dB0)
    assert missing == 0
    none = ids < 0
    assert none.any()
    np.testing.assert_array_equal(dx[none], f64(dx0)[none])
    for slot in range(5):
        r = int(t.slot_rank[slot])
        np.testing.assert_array_equal(dA[slot, r:], dA0[slot, r:])
        np.testing.assert_array_equal(dB[slot, r:], dB0[slot, r:])
    np.testing.assert_array_equal(dA[4], dA0[4])
    np.testing.assert_array_equal(dB[4], dB0[4])
    assert not np.isnan(dx).any() and not np.isnan(dA).any() and not np.isnan(dB).any()   # NaN padding never read


def test_linear_in_dy_and_in_scale():
    case = small_case(name="bwd-lin")
    dy = upstream(case)
    dx1, dA1, dB1, _ = run_backward(case, dy)
    dy2 = bits(2.0 * synth.bf16_bits_to_f64(dy))    # doubling is exact in bf16
    dx2, dA2, dB2, _ = run_backward(case, dy2)
    np.testing.assert_allclose(dx2, 2 * dx1, rtol=1e-13)
    np.testing.assert_allclose(dA2, 2 * dA1, rtol=1e-13)
    np.testing.assert_allclose(dB2, 2 * dB1, rtol=1e-13)
    t = case.table
    dx3, dA3, dB3, _ = backward.lora_backward(case.ids, t.id_to_slot, t.slot_rank, 4.0 * t.slot_scale, case.A, case.B,
                                              case.x, dy)
    np.testing.assert_allclose(dx3, 4 * dx1, rtol=1e-13)
    np.testing.assert_allclose(dA3, 4 * dA1, rtol=1e-13)


def test_not_resident_tokens_are_counted_and_skipped():
    case = small_case(name="bwd-missing")
    t = case.table
    table = t.id_to_slot.copy()
    victim = int(case.ids[case.ids >= 0][0])
    table[victim] = -1
    dy = upstream(case)
    dx, dA, dB, missing = backward.lora_backward(case.ids, table, t.slot_rank, t.slot_scale, case.A, case.B, case.x, dy)
    assert missing == int((case.ids == victim).sum())
    np.testing.assert_array_equal(dx[case.ids == victim], 0.0)

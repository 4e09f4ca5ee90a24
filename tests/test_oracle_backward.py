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


# ---- per-expert LoRA tensors (packed MoE layout) --------------------------------------
def moe_case(tag="bwd-moe-pin", T=9, K=3, E=5, num_slots=3, rank=3, d=10, n=6, proj="gate", p_none=0.2):
    batch = synth.config4_batch(T=T, E=E, K=K, num_slots=num_slots, rank=rank, p_none=p_none, tag=tag)
    return synth.config4_projection(batch, proj, d=d, n=n, tag=tag)


def run_moe_backward(c, dy, **kw):
    t = c.table
    kw.setdefault("x_row", c.x_row)
    kw.setdefault("pair_weight", c.pair_weight)
    return backward.moe_lora_backward(c.ids, c.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale, c.A, c.B, c.x,
                                      dy, **kw)


def moe_forward_loss(c, dy, x=None, A=None, B=None):
    t = c.table
    zero = np.zeros((c.T * c.K, c.n), dtype=np.uint16)
    y, _ = oracle.moe_lora_apply(c.ids, c.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                 c.A if A is None else A, c.B if B is None else B, c.x if x is None else x, zero,
                                 x_row=c.x_row, pair_weight=c.pair_weight)
    return float((y * f64(dy)).sum())


def test_moe_backward_hand_worked_pair():
    """One pair, d = 2, rank 1, n = 2, scale 2, routing weight 0.5: A = [[1], [2]], B = [[3, -1]],
    x = [1, 1] so v = 3; dy = [1, 2] so u = 3 - 2 = 1; w s = 1:
    dx = A u = [1, 2], dA = x u = [[1], [1]], dB = v dy = [[3, 6]]."""
    A = bits(np.array([[[[1.0], [2.0]]]]))          # [slot, expert, d, r]
    B = bits(np.array([[[[3.0, -1.0]]]]))           # [slot, expert, r, n]
    dx, dA, dB, missing = backward.moe_lora_backward(
        [0], np.array([[0]], np.int32), [0], [1], [2.0], A, B, bits([[1.0, 1.0]]), bits([[1.0, 2.0]]),
        pair_weight=np.array([0.5], np.float32))
    assert missing == 0
    np.testing.assert_array_equal(dx, [[1.0, 2.0]])
    np.testing.assert_array_equal(dA, [[[[1.0], [1.0]]]])
    np.testing.assert_array_equal(dB, [[[[3.0, 6.0]]]])


@pytest.mark.parametrize("proj", ["gate", "down"])
def test_moe_backward_central_differences_of_the_forward_oracle(proj):
    """As for the dense backward: L = <y, dy> through the forward MoE oracle (the C program) is linear
    in each of x, A and B, so central differences around 0 are exact.  For gate, several pairs read
    one x row: dL/dx of that row is the sum of the pairs' dx rows."""
    c = moe_case(proj=proj)
    P = c.T * c.K
    dy = synth.normal_bf16(synth.stream(c.name, "dy"), (P, c.n), 1.0)
    dx, dA, dB, _ = run_moe_backward(c, dy)
    rows = np.arange(P) if c.x_row is None else c.x_row
    rng = np.random.default_rng(11)
    h = 0.5
    for _ in range(10):
        row, col = int(rng.integers(c.x.shape[0])), int(rng.integers(c.d))
        xp, xm = c.x.copy(), c.x.copy()
        xp[row, col], xm[row, col] = bits(h).item(), bits(-h).item()
        fd = (moe_forward_loss(c, dy, x=xp) - moe_forward_loss(c, dy, x=xm)) / (2 * h)
        assert fd == pytest.approx(dx[rows == row, col].sum(), rel=1e-9, abs=1e-9)
    t = c.table
    active = [(tt, k) for tt in range(c.T) for k in range(c.K) if c.ids[tt] >= 0]
    for _ in range(12):
        tt, k = active[int(rng.integers(len(active)))]
        slot, e = int(t.id_to_slot[c.ids[tt]]), int(c.expert_ids[tt, k])
        rk = int(rng.integers(t.slot_rank[slot]))
        col = int(rng.integers(c.d))
        Ap, Am = c.A.copy(), c.A.copy()
        Ap[slot, e, col, rk], Am[slot, e, col, rk] = bits(h).item(), bits(-h).item()
        fd = (moe_forward_loss(c, dy, A=Ap) - moe_forward_loss(c, dy, A=Am)) / (2 * h)
        assert fd == pytest.approx(dA[slot, e, col, rk], rel=1e-9, abs=1e-9)
        j = int(rng.integers(c.n))
        Bp, Bm = c.B.copy(), c.B.copy()
        Bp[slot, e, rk, j], Bm[slot, e, rk, j] = bits(h).item(), bits(-h).item()
        fd = (moe_forward_loss(c, dy, B=Bp) - moe_forward_loss(c, dy, B=Bm)) / (2 * h)
        assert fd == pytest.approx(dB[slot, e, rk, j], rel=1e-9, abs=1e-9)


def test_moe_backward_one_expert_one_route_is_the_dense_backward():
    """E = K = 1 with unit weights: the packed tensors are the dense ones with A transposed."""
    case = small_case("bwd-moe-dense", p_none=0.1)
    dy = upstream(case)
    dx, dA, dB, _ = run_backward(case, dy)
    t = case.table
    A_moe = np.ascontiguousarray(case.A.transpose(0, 2, 1))[:, None]        # [slots, 1, d, r_max]
    B_moe = case.B[:, None]                                                   # [slots, 1, r_max, n]
    mdx, mdA, mdB, _ = backward.moe_lora_backward(case.ids, np.zeros((case.T, 1), np.int32), t.id_to_slot,
                                                  t.slot_rank, t.slot_scale, A_moe, B_moe, case.x, dy)
    np.testing.assert_allclose(mdx, dx, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(mdA[:, 0].transpose(0, 2, 1), dA, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(mdB[:, 0], dB, rtol=1e-12, atol=1e-12)


def test_moe_backward_masks_and_weights():
    """Ranks at or above the slot's rank and (slot, expert) blocks without pairs keep their starting
    values bit for bit; pairs of tokens without an adapter and of expert ids out of
    range keep their dx row; a constant routing weight c is the scale times c."""
    c = moe_case(tag="bwd-moe-mask", rank=2, p_none=0.3)
    P = c.T * c.K
    dy = synth.normal_bf16(synth.stream(c.name, "dy"), (P, c.n), 1.0)
    ex = c.expert_ids.copy()
    live = np.nonzero(c.ids >= 0)[0]
    ex[live[0], 0] = c.E + 3                                     # dropped pair
    t = c.table
    t.slot_rank = t.slot_rank.copy()
    t.slot_rank[0] = 1                                           # a slot padded up to r_max
    r_max = c.A.shape[3]
    used = np.zeros((t.num_slots, c.E), bool)
    for tt in live:
        for k in range(c.K):
            if 0 <= ex[tt, k] < c.E:
                used[t.id_to_slot[c.ids[tt]], ex[tt, k]] = True
    dA0 = np.full(c.A.shape, 7.0)
    dB0 = np.full(c.B.shape, -3.0)
    touch_a = np.zeros(c.A.shape, bool)
    touch_b = np.zeros(c.B.shape, bool)
    for s_ in range(t.num_slots):
        touch_a[s_, used[s_], :, :t.slot_rank[s_]] = True
        touch_b[s_, used[s_], :t.slot_rank[s_], :] = True
    dx0 = synth.normal_bf16(synth.stream(c.name, "dx0"), (P, c.d), 1.0)
    dx, dA, dB, _ = backward.moe_lora_backward(c.ids, ex, t.id_to_slot, t.slot_rank, t.slot_scale, c.A, c.B, c.x, dy,
                                               x_row=c.x_row, pair_weight=c.pair_weight, dx0=dx0, dA0=dA0, dB0=dB0)
    assert t.slot_rank.min() < r_max and not used.all()        # there is padding and there are idle blocks
    assert (dA[~touch_a] == 7.0).all() and (dB[~touch_b] == -3.0).all()
    assert (dA[touch_a] != 7.0).mean() > 0.99 and (dB[touch_b] != -3.0).mean() > 0.99
    dead = np.repeat(c.ids < 0, c.K)
    dead[live[0] * c.K] = True
    np.testing.assert_array_equal(dx[dead], f64(dx0)[dead])
    assert np.abs(dx[~dead] - f64(dx0)[~dead]).max() > 0
    const = np.full(P, 0.25, np.float32)
    a = backward.moe_lora_backward(c.ids, ex, t.id_to_slot, t.slot_rank, t.slot_scale, c.A, c.B, c.x, dy,
                                   x_row=c.x_row, pair_weight=const)
    b = backward.moe_lora_backward(c.ids, ex, t.id_to_slot, t.slot_rank, t.slot_scale * np.float32(0.25), c.A, c.B,
                                   c.x, dy, x_row=c.x_row)
    for u_, v_ in zip(a[:3], b[:3]):
        np.testing.assert_allclose(u_, v_, rtol=1e-12, atol=1e-15)

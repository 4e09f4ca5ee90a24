"""Dense shrink / expand / fused apply on the GPU against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2605_13779_b200 import synth
import parity

pytestmark = pytest.mark.gpu


def run_fused(case, y0_bits=None):
    from paper_2605_13779_b200 import binding as mb, harness
    dev = harness.upload_dense(case)
    if y0_bits is not None:
        dev.y = mb.bf16_from_bits(y0_bits)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    mb.mint_lora_apply_fused(dev.pool, dev.table, plan, dev.x, dev.y, dev.status)
    torch.cuda.synchronize()
    return harness.y_to_f64(dev.y), dev.status.cpu().numpy(), dev


def run_unfused(case):
    from paper_2605_13779_b200 import binding as mb, harness
    dev = harness.upload_dense(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    v = torch.full((case.T, case.r_max), float("nan"), dtype=torch.float32, device="cuda")
    mb.mint_lora_shrink(dev.pool, dev.table, plan, dev.x, dev.status, v=v)
    mb.mint_lora_expand(dev.pool, dev.table, plan, v, dev.y, dev.status)
    torch.cuda.synchronize()
    return harness.y_to_f64(dev.y), v.cpu().numpy().astype(np.float64), dev.status.cpu().numpy()


def check_case(case, what):
    y_ref, v_ref, missing = parity.oracle_dense(case, want_v=True)
    y_f, status, _ = run_fused(case)
    assert status[0] == 0, status
    parity.assert_close(y_f, y_ref, what + " fused")
    y_u, v_u, status = run_unfused(case)
    assert status[0] == 0, status
    parity.assert_close(y_u, y_ref, what + " shrink+expand")
    # shrink output is fully defined: zeros beyond the rank and for tokens without adapter
    np.testing.assert_allclose(v_u, v_ref, rtol=2e-4, atol=2e-4 * max(1.0, np.abs(v_ref).max()))
    assert (v_u[v_ref == 0] == 0).all()
    # rows of tokens without an adapter are untouched bit for bit
    none = case.ids < 0
    if none.any():
        np.testing.assert_array_equal(y_f[none], synth.bf16_bits_to_f64(case.y0)[none])
    # the delta itself: same case with y0 = 0, where the 5e-3 bound bites on the update
    zero = np.zeros_like(case.y0)
    y_ref0, _, _ = parity.oracle_dense(case, y0=zero)
    y_f0, _, _ = run_fused(case, y0_bits=zero)
    parity.assert_close(y_f0, y_ref0, what + " fused, y0=0")


def test_config1():
    check_case(synth.config1(), "config1")


@pytest.mark.parametrize("proj", list(synth.QWEN3_4B_PROJECTIONS))
def test_config2_projection(proj):
    batch = synth.config2_batch()
    check_case(synth.config2_projection(batch, proj), f"config2/{proj}")


def test_config3_reduced_lengths():
    """Prefill segments at one eighth of the lengths (16..128 tokens per request)."""
    batch = synth.config3_batch(len_lo=16, len_hi=128, tag="config3/small")
    check_case(synth.config3_projection(batch, 5120, 5120, tag="config3/small"), "config3/small")


def test_config3_non_contiguous_requests():
    batch = synth.config3_batch(num_requests=12, len_lo=5, len_hi=70, rank=64, bijection=False,
                                tag="config3/iid")
    check_case(synth.config3_projection(batch, 1024, 2048, tag="config3/iid"), "config3/iid")


def test_config5_full_size():
    check_case(synth.config5(), "config5")


@pytest.mark.parametrize("T,d,n,num_slots,ranks,r_max,p_none", [
    (1, 64, 64, 1, [1], 1, 0.0),
    (3, 8, 8, 2, [2, 1], 2, 0.0),
    (37, 264, 520, 6, [1, 2, 3, 5, 7, 12], 12, 0.2),
    (130, 1032, 776, 9, [1, 4, 8, 9, 16, 17, 31, 32, 3], 32, 0.1),
    (64, 2048, 1024, 3, [64, 100, 128], 128, 0.0),
    (300, 512, 512, 2, [4, 24], 24, 0.05),
    (20, 4096, 72, 20, [8] * 20, 16, 0.0),
])
def test_ragged_shapes_and_ranks(T, d, n, num_slots, ranks, r_max, p_none):
    case = synth.random_dense_case(f"gpu/ragged/{T}/{d}/{n}", T, d, n, num_slots, ranks, r_max, p_none=p_none)
    check_case(case, f"ragged T={T} d={d} n={n}")


def test_empty_batch_and_all_none():
    from paper_2605_13779_b200 import binding as mb, harness
    case = synth.random_dense_case("gpu/empty", 0, 64, 64, 2, [2, 2], 2)
    y, status, _ = run_fused(case)
    assert y.shape == (0, 64) and status[0] == 0
    case = synth.random_dense_case("gpu/allnone", 19, 64, 64, 2, [2, 2], 2, p_none=1.0)
    y, status, _ = run_fused(case)
    np.testing.assert_array_equal(y, synth.bf16_bits_to_f64(case.y0))
    assert status[0] == 0


def test_rank_padding_is_never_read():
    """Rank-r adapters in an r_max-wide slot with NaN padding equal the same
    adapters in exact-size slots."""
    wide = synth.random_dense_case("gpu/pad", 40, 256, 256, 3, [2, 3, 1], 8, p_none=0.0)
    y_wide, status, _ = run_fused(wide)
    assert status[0] == 0 and np.isfinite(y_wide).all()
    tight = synth.DenseCase("gpu/pad/tight", wide.T, wide.d, wide.n, 3, wide.table, wide.ids,
                            wide.A[:, :3].copy(), wide.B[:, :3].copy(), wide.x, wide.y0)
    y_tight, _, _ = run_fused(tight)
    np.testing.assert_array_equal(y_wide, y_tight)


def test_mixed_batch_rows_equal_isolated_rows():
    case = synth.config1()
    y_mixed, _, _ = run_fused(case)
    for a in range(4):
        sel = np.nonzero(case.ids == a)[0]
        iso = synth.DenseCase("iso", sel.size, case.d, case.n, case.r_max, case.table, case.ids[sel],
                              case.A, case.B, case.x[sel], case.y0[sel])
        y_iso, _, _ = run_fused(iso)
        # same tokens, possibly tiled differently: equal to within one bf16 rounding of the sum
        assert np.abs(y_iso - y_mixed[sel]).max() <= 2.0 ** -6


def test_fused_is_deterministic():
    case = synth.config2_projection(synth.config2_batch(), "o")
    y1, _, _ = run_fused(case)
    y2, _, _ = run_fused(case)
    np.testing.assert_array_equal(y1, y2)


def test_non_resident_tokens_are_left_untouched():
    from paper_2605_13779_b200 import binding as mb
    case = synth.config5(T=128, d=256, n=256, leave_unbound=2)
    y_ref, _, missing = parity.oracle_dense(case)
    y, status, _ = run_fused(case)
    assert missing > 0 and status[0] == mb.MINT_ERR_NOT_RESIDENT and status[1] == missing
    parity.assert_close(y, y_ref, "config5 with unbound ids")
    gone = case.table.id_to_slot[case.ids] < 0
    np.testing.assert_array_equal(y[gone], synth.bf16_bits_to_f64(case.y0)[gone])


def test_strided_activations():
    """x and y as column slices of wider buffers (row stride > width)."""
    from paper_2605_13779_b200 import binding as mb, harness
    case = synth.random_dense_case("gpu/strided", 21, 128, 192, 3, [4, 4, 2], 4, p_none=0.1)
    dev = harness.upload_dense(case)
    xw = torch.zeros(case.T, 128 + 64, dtype=torch.bfloat16, device="cuda")
    yw = torch.zeros(case.T, 192 + 8, dtype=torch.bfloat16, device="cuda")
    xw[:, :128] = dev.x
    yw[:, :192] = dev.y
    yw[:, 192:] = 5.0
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    mb.mint_lora_apply_fused(dev.pool, dev.table, plan, xw[:, :128], yw[:, :192], dev.status)
    torch.cuda.synchronize()
    y_ref, _, _ = parity.oracle_dense(case)
    parity.assert_close(harness.y_to_f64(yw[:, :192]), y_ref, "strided")
    assert (yw[:, 192:] == 5.0).all()


def test_grouped_call_equals_separate_calls():
    """q, k and v read the same x: one grouped call gives the same bits as three calls."""
    from paper_2605_13779_b200 import binding as mb, harness
    batch = synth.config2_batch()
    cases = [synth.config2_projection(batch, p) for p in ("q", "k", "v")]
    devs = [harness.upload_dense(c) for c in cases]
    table, status = devs[0].table, devs[0].status
    plan = mb.mint_lora_plan(table, devs[0].ids, status)
    x = devs[0].x
    sep = []
    for dv in devs:
        y = dv.y.clone()
        mb.mint_lora_apply_fused(dv.pool, table, plan, x, y, status)
        sep.append(y)
    ws = [mb.new_workspace(dv.pool, batch.T) for dv in devs]
    group = mb.ApplyGroup([(dv.pool, x, dv.y, w) for dv, w in zip(devs, ws)])
    mb.mint_lora_apply_fused_grouped(group, table, plan, status)
    mb.mint_lora_apply_fused_grouped(group, table, plan, status)     # workspaces are reusable as they are
    torch.cuda.synchronize()
    assert status[0].item() == 0
    for dv, c, y1 in zip(devs, cases, sep):
        once = harness.y_to_f64(y1)
        c2 = synth.DenseCase(c.name, c.T, c.d, c.n, c.r_max, c.table, c.ids, c.A, c.B, cases[0].x, c.y0)
        y_ref, _, _ = parity.oracle_dense(c2)
        parity.assert_close(once, y_ref, c.name)
        # second application on top of the first: y0 + 2 delta within two roundings
        twice = harness.y_to_f64(dv.y)
        delta = y_ref - synth.bf16_bits_to_f64(c.y0)
        assert np.abs(twice - (y_ref + delta)).max() <= 6e-2


def dense_segment_case(name, lengths, adapters, ranks, d, n, r_max):
    """Requests of the given lengths, request i bound to adapters[i]; tokens of a
    request are contiguous, an adapter may own several requests."""
    num_slots = len(ranks)
    table = synth.identity_table(num_slots, np.asarray(ranks, dtype=np.int32), 2.0)
    ids = np.repeat(np.asarray(adapters, dtype=np.int64), np.asarray(lengths, dtype=np.int64))
    T = int(ids.shape[0])
    A, B = synth.dense_pool(synth.stream(name, "pool"), table, r_max, d, n)
    x = synth.normal_bf16(synth.stream(name, "x"), (T, d), 1.0)
    y0 = synth.normal_bf16(synth.stream(name, "y0"), (T, n), 1.0)
    return synth.DenseCase(name, T, d, n, r_max, table, ids, A, B, x, y0)


def test_dense_segments_take_the_tensor_core_kernels():
    """A batch of more than 4096 tokens with segments of 128 tokens and more: their
    shrink and their expand run on the tcgen05 kernels (full and ragged 128-row tiles, ranks that are
    not multiples of 16, an adapter whose tokens are not contiguous), short segments
    and tokens without adapter stay on the streamed path."""
    lengths = [700, 130, 128, 127, 300, 5, 1, 1000, 64, 513, 256, 129, 3, 640, 384, 40]
    adapters = [0, 1, 2, 3, 4, 5, 6, 7, 8, 0, 9, 10, -1, 11, 12, 6]
    ranks = [64, 16, 8, 33, 1, 4, 32, 64, 16, 48, 5, 64, 17]
    case = dense_segment_case("gpu/dense-tc", lengths, adapters, ranks, d=1032, n=520, r_max=64)
    assert case.T >= 4096
    check_case(case, "dense segments")


def test_dense_segments_grouped_projections_of_different_widths():
    """Two projections of different widths in one grouped call over a batch with
    dense segments: both take one range of columns per 128-row tile in the
    tensor-core expand, the wide one with a ragged last 128-column chunk (n = 2184);
    the ranges of the two lie end to end in the grid.  (Several column
    ranges per tile: test_dense_segments_wide_output_takes_several_column_ranges.)"""
    from paper_2605_13779_b200 import binding as mb, harness
    lengths = [900, 128, 257, 60, 1100, 131, 2, 640, 512, 400]
    adapters = [0, 1, 2, 3, 4, 5, 3, 0, 6, -1]
    ranks = [64, 24, 16, 8, 40, 1, 64]
    wide = dense_segment_case("gpu/dense-tc/wide", lengths, adapters, ranks, d=520, n=2184, r_max=64)
    narrow = dense_segment_case("gpu/dense-tc/narrow", lengths, adapters, ranks, d=520, n=264, r_max=64)
    assert wide.T >= 4096
    devs = [harness.upload_dense(c) for c in (wide, narrow)]
    table, status = devs[0].table, devs[0].status
    plan = mb.mint_lora_plan(table, devs[0].ids, status)
    ws = [mb.new_workspace(dv.pool, wide.T) for dv in devs]
    group = mb.ApplyGroup([(dv.pool, dv.x, dv.y, w) for dv, w in zip(devs, ws)])
    mb.mint_lora_apply_fused_grouped(group, table, plan, status)
    torch.cuda.synchronize()
    assert status[0].item() == 0
    for dv, c in zip(devs, (wide, narrow)):
        y_ref, _, _ = parity.oracle_dense(c)
        parity.assert_close(harness.y_to_f64(dv.y), y_ref, c.name)
        none = c.ids < 0
        np.testing.assert_array_equal(harness.y_to_f64(dv.y)[none], synth.bf16_bits_to_f64(c.y0)[none])


def test_dense_segments_config3_shape_sampled():
    """One config-3 projection at full size on the tensor-core shrink, checked on sampled rows."""
    from paper_2605_13779_b200 import binding as mb, harness
    batch = synth.config3_batch()
    case = synth.config3_projection(batch, 5120, 5120)
    y, status, _ = run_fused(case)
    assert status[0] == 0, status
    rng = synth.stream("gpu/dense-tc/sample")
    rows = np.sort(rng.choice(case.T, size=96, replace=False))
    # include the first and last token of some requests (tile edges)
    edges = np.cumsum(batch.lengths)
    rows = np.unique(np.concatenate([rows, edges[:8] - 1, edges[:8] % case.T]))
    y_ref, _, _ = parity.oracle_dense(case, rows=rows)
    parity.assert_close(y[rows], y_ref, "config3 sampled rows")


def run_fused_rows(case, rows, y0_zero=False):
    """The fused apply at full size; only the given rows of y come back to the host."""
    from paper_2605_13779_b200 import binding as mb, harness
    dev = harness.upload_dense(case)
    if y0_zero:
        dev.y.zero_()
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    mb.mint_lora_apply_fused(dev.pool, dev.table, plan, dev.x, dev.y, dev.status)
    torch.cuda.synchronize()
    idx = torch.from_numpy(np.asarray(rows, dtype=np.int64)).cuda()
    return harness.y_to_f64(dev.y[idx]), dev.status.cpu().numpy()


SPLIT_LENGTHS = [700, 130, 128, 127, 300, 5, 1, 1000, 64, 513, 256, 129, 3, 640, 384, 40]
SPLIT_ADAPTERS = [0, 1, 2, 3, 4, 5, 6, 7, 8, 0, 9, 10, -1, 11, 12, 6]
SPLIT_RANKS = [64, 16, 8, 33, 1, 4, 32, 64, 16, 48, 5, 64, 17]


@pytest.mark.parametrize("d,parts", [(10240, 2), (15360, 3), (25600, 4), (20488, 4)])
def test_dense_segments_wide_input_is_split_over_several_ctas(d, parts):
    """Input widths of 10240 and more: the tensor-core shrink of a 128-row tile is
    split over 2, 3 or 4 CTAs, each over its share of the columns of d, and the
    expand adds their parts.  Full and ragged 128-row tiles, ranks that are not
    multiples of 16, a last 64-column chunk that is not full (d = 20488)."""
    case = dense_segment_case(f"gpu/dense-tc/split/{d}", SPLIT_LENGTHS, SPLIT_ADAPTERS, SPLIT_RANKS,
                              d=d, n=264, r_max=64)
    assert case.T >= 4096
    check_case(case, f"dense segments d={d} ({parts} parts)")


@pytest.mark.parametrize("n", [25600, 24584, 40968])
def test_dense_segments_wide_output_takes_several_column_ranges(n):
    """The tensor-core expand gives a 128-row tile one CTA per range of at most 16384
    columns, the ranges of a projection equally wide: n = 25600 is two ranges of 12800,
    n = 24584 two of 12416 and 12168 columns, n = 40968 three, and the last 128-column
    chunk of the last two holds 8 columns (a ragged chunk)."""
    case = dense_segment_case(f"gpu/dense-tc/wide-n/{n}", SPLIT_LENGTHS, SPLIT_ADAPTERS, SPLIT_RANKS,
                              d=520, n=n, r_max=64)
    y_ref, _, _ = parity.oracle_dense(case)
    y, status, _ = run_fused(case)
    assert status[0] == 0, status
    parity.assert_close(y, y_ref, f"dense segments n={n}")
    none = case.ids < 0
    np.testing.assert_array_equal(y[none], synth.bf16_bits_to_f64(case.y0)[none])
    zero = np.zeros_like(case.y0)
    y_ref0, _, _ = parity.oracle_dense(case, y0=zero)
    y0, _, _ = run_fused(case, y0_bits=zero)
    parity.assert_close(y0, y_ref0, f"dense segments n={n}, y0=0")


@pytest.mark.parametrize("d,n", [(5120, 25600), (25600, 5120)])
def test_config3_wide_projections_full_size_sampled(d, n):
    """The up (5120 -> 25600) and down (25600 -> 5120) projections of the 32B-dense
    segmented prefill at full size (about 18k tokens), checked on sampled rows that
    include the first and last token of requests (edges of 128-row tiles), with
    the preset y and with y = 0."""
    batch = synth.config3_batch()
    case = synth.config3_projection(batch, d, n)
    rng = synth.stream("gpu/dense-tc/sample", d, n)
    rows = np.sort(rng.choice(case.T, size=64, replace=False))
    edges = np.cumsum(batch.lengths)
    rows = np.unique(np.concatenate([rows, edges[:8] - 1, edges[:8] % case.T, edges[:4] - 129, edges[:4] - 128]))
    rows = rows[(rows >= 0) & (rows < case.T)]
    for y0_zero in (False, True):
        y, status = run_fused_rows(case, rows, y0_zero=y0_zero)
        assert status[0] == 0, status
        y_ref, _, _ = parity.oracle_dense(case, rows=rows, y0=np.zeros_like(case.y0) if y0_zero else None)
        parity.assert_close(y, y_ref, f"config3 {d}->{n} sampled rows y0_zero={y0_zero}")

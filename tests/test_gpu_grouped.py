"""Grouped fused calls against the fp64 oracle: the call shapes the benchmark times
(all seven projections of the 4B-dense decode layer in one call; the four calls
a transformer layer's data dependencies allow) and groups of equal-width
projections, where one tile meets many shrink lanes."""
import numpy as np
import pytest
import torch

from paper_2605_13779_b200 import synth
import parity

pytestmark = pytest.mark.gpu

STAGES = (("q", "k", "v"), ("o",), ("gate", "up"), ("down",))


def run_grouped(cases, groups, y0_zero=False, repeat=1):
    """Uploads the cases (one shared table and plan), applies them in the given
    groups of indices, returns the list of y as fp64 and the status words."""
    from paper_2605_13779_b200 import binding as mb, harness
    table = harness.upload_table(cases[0].table)
    devs = [harness.upload_dense(c, table=table) for c in cases]
    for i in range(1, len(cases)):   # projections with the same input read one tensor
        if cases[i].x.shape == cases[i - 1].x.shape and np.array_equal(cases[i].x, cases[i - 1].x):
            devs[i].x = devs[i - 1].x
    if y0_zero:
        for dv in devs:
            dv.y.zero_()
    status = devs[0].status
    plan = mb.mint_lora_plan(table, devs[0].ids, status)
    ws = [mb.new_workspace(dv.pool, cases[0].T) for dv in devs]
    for w in ws:
        w.fill_(0xFF)       # the workspace needs no initialisation: NaN patterns must never reach y
    for _ in range(repeat):
        for g in groups:
            grp = mb.ApplyGroup([(devs[i].pool, devs[i].x, devs[i].y, ws[i]) for i in g])
            mb.mint_lora_apply_fused_grouped(grp, table, plan, status)
    torch.cuda.synchronize()
    return [harness.y_to_f64(dv.y) for dv in devs], status.cpu().numpy()


def check_groups(cases, groups, what):
    for y0_zero in (False, True):
        ys, status = run_grouped(cases, groups, y0_zero=y0_zero)
        assert status[0] == 0, status
        for c, y in zip(cases, ys):
            y0 = np.zeros_like(c.y0) if y0_zero else None
            y_ref, _, _ = parity.oracle_dense(c, y0=y0)
            parity.assert_close(y, y_ref, f"{what} {c.name} y0_zero={y0_zero}")
            none = c.ids < 0
            if none.any():
                start = np.zeros(c.y0.shape) if y0_zero else synth.bf16_bits_to_f64(c.y0)
                np.testing.assert_array_equal(y[none], start[none])


def config2_cases():
    batch = synth.config2_batch()
    return [synth.config2_projection(batch, p) for p in synth.QWEN3_4B_PROJECTIONS]


def test_config2_whole_layer_in_one_call():
    """The benchmark's default call: seven projections of three different input
    widths and five different output widths side by side in one launch pair."""
    cases = config2_cases()
    check_groups(cases, [list(range(7))], "layer call")


def test_config2_stage_calls():
    """q,k,v | o | gate,up | down: the four calls a decoder layer can issue."""
    cases = config2_cases()
    names = list(synth.QWEN3_4B_PROJECTIONS)
    groups = [[names.index(p) for p in st] for st in STAGES]
    check_groups(cases, groups, "stage calls")


def test_config2_layer_call_with_tokens_without_adapter():
    batch = synth.config2_batch(tag="config2/none")
    batch.ids[::7] = -1
    cases = [synth.config2_projection(batch, p, tag="config2/none") for p in synth.QWEN3_4B_PROJECTIONS]
    check_groups(cases, [list(range(7))], "layer call with none")


def equal_width_cases(count, T, rank, d=2560, n=64, num_slots=1, tag="gpu/equal", same_x=1, ranks=None):
    """same_x: runs of that many consecutive projections read the same x."""
    ranks = np.full(num_slots, rank, dtype=np.int32) if ranks is None else np.asarray(ranks, dtype=np.int32)
    table = synth.identity_table(num_slots, ranks, 2.0)
    ids = (np.arange(T) % num_slots).astype(np.int64)
    cases = []
    for i in range(count):
        name = f"{tag}/{count}/{T}/{rank}/{i}"
        A, B = synth.dense_pool(synth.stream(name, "pool"), table, rank, d, n)
        x = synth.normal_bf16(synth.stream(f"{tag}/{count}/{T}/{rank}/{i // same_x}", "x"), (T, d), 1.0)
        y0 = synth.normal_bf16(synth.stream(name, "y0"), (T, n), 1.0)
        cases.append(synth.DenseCase(name, T, d, n, rank, table, ids, A, B, x, y0))
    return cases


@pytest.mark.parametrize("count,T,rank", [(8, 1, 8), (8, 32, 32), (7, 32, 32), (7, 1, 8), (8, 20, 16), (8, 5, 1)])
def test_equal_width_projections_share_one_tile(count, T, rank):
    """Many projections of the same width over a one-adapter batch: the single
    tile of the plan is cut into far more shrink shares than one projection
    meets, and every projection still has to find exactly its own."""
    cases = equal_width_cases(count, T, rank)
    check_groups(cases, [list(range(count))], f"equal widths x{count} T={T} r={rank}")


@pytest.mark.parametrize("count,T,num_slots,rank", [(8, 64, 3, 16), (6, 200, 20, 8)])
def test_equal_width_projections_several_adapters(count, T, num_slots, rank):
    cases = equal_width_cases(count, T, rank, d=1024, n=512, num_slots=num_slots, tag="gpu/equal-multi")
    check_groups(cases, [list(range(count))], f"equal widths x{count} T={T} slots={num_slots}")


def test_grouped_call_twice_on_one_workspace():
    """Two grouped calls back to back reuse the workspaces as the first left them."""
    cases = config2_cases()[:3]
    ys, status = run_grouped(cases, [[0, 1, 2]], repeat=2)
    assert status[0] == 0
    for c, y in zip(cases, ys):
        y_ref, _, _ = parity.oracle_dense(c)
        delta = y_ref - synth.bf16_bits_to_f64(c.y0)
        assert np.abs(y - (y_ref + delta)).max() <= 6e-2


@pytest.mark.parametrize("count,same_x,T,num_slots,ranks,r_max", [
    (3, 3, 40, 4, [8, 1, 16, 32], 32),      # q, k, v: three pools, one x
    (2, 2, 33, 3, [16, 5, 1], 16),          # gate, up
    (5, 2, 70, 5, [32, 8, 1, 16, 3], 32),   # pairs, then one projection on its own
    (7, 3, 16, 2, [1, 1], 8),               # rank 1 only: the FMA path of every member
    (8, 4, 50, 3, [8, 16, 2], 16),          # runs of four: groups of three and one
])
def test_projections_that_read_the_same_x(count, same_x, T, num_slots, ranks, r_max):
    """Items of a grouped call may read the same x tensor (q, k, v; gate, up)."""
    cases = equal_width_cases(count, T, r_max, d=1032, n=264, num_slots=num_slots, tag="gpu/same-x",
                              same_x=same_x, ranks=ranks)
    check_groups(cases, [list(range(count))], f"same x: {count} items in runs of {same_x}")


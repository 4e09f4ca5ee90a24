"""LoRA backward over padded slots on the GPU against the fp64 oracle.

Tolerances: dx is a bf16 tensor updated like y in the forward path, so the forward bar holds
(max |delta| <= 3e-2, relative Frobenius <= 5e-3 over the full tensor, and again with dx0 = 0);
dA and dB are fp32 sums of fp32 products of exact bf16 inputs and of u, v that carry fp32
accumulation over d or n (relative error about 1e-6 sqrt(width) at worst): relative Frobenius
<= 1e-4 per slot tensor, and the untouched parts (padding rows, slots without tokens) bit for bit."""
import numpy as np
import pytest
import torch

from oracle import backward
from paper_2605_13779_b200 import synth
import parity

pytestmark = pytest.mark.gpu


def run_backward(case, dy, dx0_zero=False, want_dx=True, want_grads=True, repeat=1):
    from paper_2605_13779_b200 import binding as mb, harness
    dev = harness.upload_dense(case)
    dyd = mb.bf16_from_bits(dy)
    dx0 = np.zeros_like(case.x) if dx0_zero else synth.normal_bf16(synth.stream(case.name, "dx0"), case.x.shape, 1.0)
    dx = mb.bf16_from_bits(dx0) if want_dx else None
    dA0 = synth.stream(case.name, "dA0").standard_normal(case.A.shape).astype(np.float32)
    dB0 = synth.stream(case.name, "dB0").standard_normal(case.B.shape).astype(np.float32)
    dA = torch.from_numpy(dA0.copy()).cuda() if want_grads else None
    dB = torch.from_numpy(dB0.copy()).cuda() if want_grads else None
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    ws = mb.new_backward_workspace(dev.pool, case.T)
    ws.fill_(0xFF)   # the workspace needs no initialisation
    for _ in range(repeat):
        mb.mint_lora_backward(dev.pool, dev.table, plan, dev.x, dyd, dev.status, dx=dx, dA=dA, dB=dB, workspace=ws)
    torch.cuda.synchronize()
    out = {"status": dev.status.cpu().numpy(), "dx0": dx0, "dA0": dA0, "dB0": dB0}
    if want_dx:
        out["dx"] = harness.y_to_f64(dx)
    if want_grads:
        out["dA"] = dA.cpu().numpy().astype(np.float64)
        out["dB"] = dB.cpu().numpy().astype(np.float64)
    return out


def oracle_backward(case, dy, dx0, dA0, dB0):
    t = case.table
    return backward.lora_backward(case.ids, t.id_to_slot, t.slot_rank, t.slot_scale, case.A, case.B, case.x, dy,
                                  dx0=dx0, dA0=dA0, dB0=dB0)


def check_grads(got, ref, start, case, what):
    t = case.table
    slots = t.id_to_slot[case.ids[case.ids >= 0]]
    used = set(int(s) for s in slots[slots >= 0])
    for slot in range(t.num_slots):
        r = int(t.slot_rank[slot])
        if slot not in used:
            np.testing.assert_array_equal(got[slot], start[slot].astype(np.float64), err_msg=f"{what}: empty slot {slot}")
            continue
        np.testing.assert_array_equal(got[slot, r:], start[slot, r:].astype(np.float64),
                                      err_msg=f"{what}: padding rows of slot {slot}")
        delta_ref = ref[slot, :r] - start[slot, :r]
        delta_got = got[slot, :r] - start[slot, :r]
        denom = np.linalg.norm(delta_ref)
        err = np.linalg.norm(delta_got - delta_ref)
        # (the update itself: the fp32 starting values contribute half an ulp of the sum each)
        ulp = 6e-8 * np.linalg.norm(ref[slot, :r])
        assert err <= 1e-4 * denom + 2 * ulp, f"{what}: slot {slot} rel {err / max(denom, 1e-30):.3e}"


def check_case(case, what):
    dy = synth.normal_bf16(synth.stream(case.name, "dy"), (case.T, case.n), 1.0)
    for dx0_zero in (False, True):
        got = run_backward(case, dy, dx0_zero=dx0_zero)
        assert got["status"][0] == 0, got["status"]
        dx_ref, dA_ref, dB_ref, _ = oracle_backward(case, dy, got["dx0"], got["dA0"], got["dB0"])
        parity.assert_close(got["dx"], dx_ref, f"{what} dx dx0_zero={dx0_zero}")
        none = case.ids < 0
        if none.any():
            np.testing.assert_array_equal(got["dx"][none], synth.bf16_bits_to_f64(got["dx0"])[none])
        check_grads(got["dA"], dA_ref, got["dA0"], case, what + " dA")
        check_grads(got["dB"], dB_ref, got["dB0"], case, what + " dB")


def test_config1_backward():
    check_case(synth.config1(), "config1")


@pytest.mark.parametrize("proj", ["q", "o", "down"])
def test_config2_projection_backward(proj):
    """Decode batch of the 4B-dense setting: 47 adapters of ranks 1, 8, 16, 32 in slots of 32."""
    batch = synth.config2_batch()
    check_case(synth.config2_projection(batch, proj), f"config2/{proj}")


@pytest.mark.parametrize("T,d,n,num_slots,ranks,r_max,p_none", [
    (1, 8, 8, 1, [1], 1, 0.0),
    (37, 72, 40, 3, [3, 1, 2], 4, 0.2),
    (130, 520, 264, 5, [8, 16, 5, 1, 12], 16, 0.1),
    (300, 1032, 2056, 4, [32, 17, 64, 40], 64, 0.05),
    (64, 4104, 520, 2, [20, 1], 24, 0.0),
])
def test_ragged_shapes_and_ranks_backward(T, d, n, num_slots, ranks, r_max, p_none):
    case = synth.random_dense_case(f"gpu/bwd/{T}/{d}/{n}", T, d, n, num_slots, ranks, r_max, p_none=p_none)
    check_case(case, f"ragged {T}x{d}x{n}")


def test_long_segments_backward():
    """Segments of hundreds of tokens (prefill-shaped): the token loop of the weight gradient runs
    over several batches; T >= 4096 also sends dx through the tensor-core kernels."""
    batch = synth.config3_batch(num_requests=10, len_lo=300, len_hi=900, rank=64, tag="gpu/bwd/long")
    case = synth.config3_projection(batch, d=1024, n=520, tag="gpu/bwd/long")
    assert case.T >= 4096
    check_case(case, "long segments")


def test_frozen_adapters_and_no_input_gradient():
    """dA/dB omitted (frozen adapters): only dx; dx omitted: only the weight gradients."""
    case = synth.random_dense_case("gpu/bwd/partial", 50, 264, 136, 3, [4, 8, 2], 8, p_none=0.1)
    dy = synth.normal_bf16(synth.stream(case.name, "dy"), (case.T, case.n), 1.0)
    full = run_backward(case, dy)
    only_dx = run_backward(case, dy, want_grads=False)
    only_w = run_backward(case, dy, want_dx=False)
    np.testing.assert_array_equal(only_dx["dx"], full["dx"])
    # (a call that wants everything shares the shrink of dy between dA and dx, so its lanes cut the columns
    # elsewhere than those of a call for the weight gradients alone: equal up to fp32 summation order)
    np.testing.assert_allclose(only_w["dA"] - full["dA0"], full["dA"] - full["dA0"], rtol=1e-4, atol=1e-5)
    np.testing.assert_allclose(only_w["dB"] - full["dB0"], full["dB"] - full["dB0"], rtol=1e-4, atol=1e-5)
    dy_ref = oracle_backward(case, dy, full["dx0"], full["dA0"], full["dB0"])
    check_grads(only_w["dA"], dy_ref[1], full["dA0"], case, "weights only dA")
    check_grads(only_w["dB"], dy_ref[2], full["dB0"], case, "weights only dB")
    parity.assert_close(only_dx["dx"], dy_ref[0], "dx only")


def test_backward_is_deterministic_and_accumulates():
    case = synth.random_dense_case("gpu/bwd/det", 90, 520, 264, 4, [8, 3, 16, 1], 16, p_none=0.1)
    dy = synth.normal_bf16(synth.stream(case.name, "dy"), (case.T, case.n), 1.0)
    a = run_backward(case, dy)
    b = run_backward(case, dy)
    for k in ("dx", "dA", "dB"):
        np.testing.assert_array_equal(a[k], b[k])
    twice = run_backward(case, dy, repeat=2)
    dx_ref, dA_ref, dB_ref, _ = oracle_backward(case, dy, a["dx0"], a["dA0"], a["dB0"])
    # two calls add the gradient twice
    np.testing.assert_allclose(twice["dA"] - a["dA0"], 2 * (dA_ref - a["dA0"]), rtol=2e-4, atol=1e-5)
    np.testing.assert_allclose(twice["dB"] - a["dB0"], 2 * (dB_ref - a["dB0"]), rtol=2e-4, atol=1e-5)


def test_grouped_backward_of_a_whole_layer():
    """The seven projections of the 4B-dense decode layer in one grouped call (as the benchmark issues it);
    one of them with frozen adapters, one without an input gradient."""
    from paper_2605_13779_b200 import binding as mb, harness
    batch = synth.config2_batch()
    cases = [synth.config2_projection(batch, p) for p in synth.QWEN3_4B_PROJECTIONS]
    table = harness.upload_table(cases[0].table)
    devs = [harness.upload_dense(c, table=table) for c in cases]
    status = devs[0].status
    plan = mb.mint_lora_plan(table, devs[0].ids, status)
    items, keep = [], []
    for i, (c, dv) in enumerate(zip(cases, devs)):
        dy = synth.normal_bf16(synth.stream(c.name, "dy"), (c.T, c.n), 1.0)
        dx0 = synth.normal_bf16(synth.stream(c.name, "dx0"), c.x.shape, 1.0)
        dx = None if i == 2 else mb.bf16_from_bits(dx0)
        frozen = i == 4
        dA = None if frozen else torch.zeros(c.A.shape, dtype=torch.float32, device="cuda")
        dB = None if frozen else torch.zeros(c.B.shape, dtype=torch.float32, device="cuda")
        ws = mb.new_backward_workspace(dv.pool, c.T)
        ws.fill_(0xFF)
        items.append((dv.pool, dv.x, mb.bf16_from_bits(dy), dx, dA, dB, ws))
        keep.append((dy, dx0))
    mb.mint_lora_backward_grouped(mb.BackwardGroup(items), table, plan, status)
    torch.cuda.synchronize()
    assert status.cpu().numpy()[0] == 0
    for c, (pool, x, dyd, dx, dA, dB, ws), (dy, dx0) in zip(cases, items, keep):
        dx_ref, dA_ref, dB_ref, _ = oracle_backward(c, dy, dx0, None, None)
        if dx is not None:
            parity.assert_close(harness.y_to_f64(dx), dx_ref, f"grouped {c.name} dx")
        if dA is not None:
            zero = np.zeros(c.A.shape, dtype=np.float32)
            check_grads(dA.cpu().numpy().astype(np.float64), dA_ref, zero, c, f"grouped {c.name} dA")
            check_grads(dB.cpu().numpy().astype(np.float64), dB_ref, np.zeros(c.B.shape, dtype=np.float32), c,
                        f"grouped {c.name} dB")

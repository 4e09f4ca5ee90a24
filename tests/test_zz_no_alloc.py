"""The fused apply with the library's built-in workspace (for callers that
cannot allocate device memory: plugins inside an engine that owns all of it,
allocation-free hot paths, fixed memory budgets) gives the same output as the
ordinary entry point, on two calls in a row that share that workspace."""
import numpy as np
import pytest
import torch

from paper_2605_13779_b200 import synth
import parity

pytestmark = pytest.mark.gpu


def test_static_workspace_matches_the_ordinary_entry_point_twice_in_a_row():
    from paper_2605_13779_b200 import binding as mb, harness
    cases = [synth.config1(),
             synth.random_dense_case("gpu/noalloc", 130, 1032, 776, 9, [1, 4, 8, 9, 16, 17, 31, 32, 3], 32, p_none=0.1)]
    outs = []
    for case in cases:                      # two calls in a row through the built-in workspace
        dev = harness.upload_dense(case)
        plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
        y_ref_entry = dev.y.clone()
        before = torch.cuda.memory_allocated()
        mb.mint_lora_apply_fused_static(dev.pool, dev.table, plan, dev.x, dev.y, dev.status)
        assert torch.cuda.memory_allocated() == before          # the binding allocated nothing either
        outs.append((case, dev, plan, y_ref_entry))
    torch.cuda.synchronize()
    for case, dev, plan, y_other in outs:
        assert dev.status[0].item() == 0
        mb.mint_lora_apply_fused(dev.pool, dev.table, plan, dev.x, y_other, dev.status)
        torch.cuda.synchronize()
        got, want = harness.y_to_f64(dev.y), harness.y_to_f64(y_other)
        parity.assert_close(got, want, case.name + " static vs ordinary entry point")
        y_ref, _, _ = parity.oracle_dense(case)
        parity.assert_close(got, y_ref, case.name + " static vs oracle")


def test_static_workspace_refuses_batches_beyond_its_size():
    from paper_2605_13779_b200 import binding as mb, harness
    case = synth.random_dense_case("gpu/noalloc/big", 64, 64, 64, 2, [64, 64], 64, p_none=0.0)
    dev = harness.upload_dense(case)
    # a plan for far more tokens than the built-in workspace can serve
    T = 200000
    ids = torch.zeros(T, dtype=torch.int64, device="cuda")
    plan = mb.mint_lora_plan(dev.table, ids, dev.status)
    assert mb.mint_lora_apply_workspace_bytes(dev.pool, T) > mb.MINT_STATIC_WORKSPACE_BYTES
    x = torch.zeros(T, 64, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(T, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mb.MintError) as e:
        mb.mint_lora_apply_fused_static(dev.pool, dev.table, plan, x, y, dev.status)
    assert e.value.status == mb.MINT_ERR_WORKSPACE_TOO_SMALL
    torch.cuda.synchronize()
    assert (y == 0).all()

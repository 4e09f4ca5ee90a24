"""The sharded apply with the CUDA binding behind the driver: two (or four) ranks'
shards run one after the other on the one GPU, the exchange of the partial v is
a sum on the host side of the test."""
import numpy as np
import pytest
import torch

from paper_2605_13779_b200 import sharding, synth
import parity

pytestmark = pytest.mark.gpu


def gpu_fused(case):
    from paper_2605_13779_b200 import binding as mb, harness
    dev = harness.upload_dense(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    mb.mint_lora_apply_fused(dev.pool, dev.table, plan, dev.x, dev.y, dev.status)
    torch.cuda.synchronize()
    assert dev.status[0].item() == 0
    return harness.y_to_f64(dev.y)


def gpu_shrink(case):
    from paper_2605_13779_b200 import binding as mb, harness
    dev = harness.upload_dense(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    v = mb.mint_lora_shrink(dev.pool, dev.table, plan, dev.x, dev.status)
    torch.cuda.synchronize()
    return v.cpu().numpy()


def gpu_expand(case, v):
    from paper_2605_13779_b200 import binding as mb, harness
    dev = harness.upload_dense(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    mb.mint_lora_expand(dev.pool, dev.table, plan, torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32)).cuda(),
                        dev.y, dev.status)
    torch.cuda.synchronize()
    return harness.y_to_f64(dev.y)


@pytest.mark.parametrize("world", [2, 4])
def test_column_and_row_parallel_projections(world):
    batch = synth.config2_batch()
    case = synth.config2_projection(batch, "o")        # 4096 -> 2560
    y_ref, _, _ = parity.oracle_dense(case)
    cols = [sharding.apply_column_parallel(gpu_fused, case, world, r) for r in range(world)]
    parity.assert_close(sharding.reassemble_columns(cols, case.n), y_ref, f"column-parallel x{world}")
    partial = [gpu_shrink(sharding.row_parallel_shard(case, world, r)) for r in range(world)]
    total = np.sum(np.stack(partial).astype(np.float64), axis=0)       # the all-reduce of v
    for r in range(world):
        y = sharding.apply_row_parallel(lambda c: partial[r], gpu_expand, lambda v: total, case, world, r)
        parity.assert_close(y, y_ref, f"row-parallel x{world} rank {r}")


def test_expert_parallel_moe():
    from paper_2605_13779_b200 import binding as mb, harness
    batch = synth.config4_batch(T=256)
    case = synth.config4_projection(batch, "gate")
    y_ref, _ = parity.oracle_moe(case)
    y = np.full_like(y_ref, np.nan)
    for rank in range(4):
        local, pairs = sharding.expert_parallel_shard(case, 4, rank)
        dev = harness.upload_moe(local)
        plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status, expert_ids=dev.expert_ids, num_experts=local.E)
        mb.mint_moe_lora_apply(dev.pool, dev.table, plan, dev.x, dev.y, dev.status)
        torch.cuda.synchronize()
        assert dev.status[0].item() == 0
        y[pairs] = harness.y_to_f64(dev.y)
    parity.assert_close(y, y_ref, "expert-parallel x4")

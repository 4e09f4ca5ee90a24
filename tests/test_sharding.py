"""Tensor-parallel / expert-parallel placement of the apply: the partition
arithmetic, and two gloo ranks on the CPU whose sharded results reassemble to
the unsharded oracle (the arithmetic of each shard is the oracle's here; on a
GPU the same driver is handed the CUDA binding, tests/test_gpu_sharding.py)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import oracle
from paper_2605_13779_b200 import sharding, synth


@pytest.mark.parametrize("width,world", [(2560, 2), (1024, 4), (9728, 8), (24, 5), (8, 3), (4096, 16)])
def test_split_range_tiles_the_width_in_multiples_of_8(width, world):
    edges = [sharding.split_range(width, world, r) for r in range(world)]
    assert edges[0][0] == 0 and edges[-1][1] == width
    for (a0, a1), (b0, b1) in zip(edges, edges[1:]):
        assert a1 == b0
    sizes = [hi - lo for lo, hi in edges]
    assert all(s % 8 == 0 for s in sizes) and max(sizes) - min(sizes) <= 8
    assert sizes == sorted(sizes, reverse=True)


def oracle_apply(case):
    t = case.table
    return oracle.lora_apply(case.ids, t.id_to_slot, t.slot_rank, t.slot_scale, case.A, case.B, case.x, case.y0)[0]


def oracle_shrink(case):
    t = case.table
    zero_b = np.zeros_like(case.B)
    return oracle.lora_apply(case.ids, t.id_to_slot, t.slot_rank, t.slot_scale, case.A, zero_b, case.x, case.y0,
                             want_v=True)[1]


def oracle_expand(case, v):
    """y0 + s * v . B with the oracle's own loops: v enters as x of a rank-r 'identity' shrink."""
    t = case.table
    S, r_max, n = case.B.shape
    y = synth.bf16_bits_to_f64(case.y0).copy()
    B = synth.bf16_bits_to_f64(case.B)
    for tok in range(case.T):
        cid = case.ids[tok]
        if cid < 0 or t.id_to_slot[cid] < 0:
            continue
        s = t.id_to_slot[cid]
        r = t.slot_rank[s]
        y[tok] += float(t.slot_scale[s]) * (v[tok, :r] @ B[s, :r, :])
    return y


def the_case():
    return synth.random_dense_case("sharding/dense", 23, 72, 88, 4, [2, 5, 1, 8], 8, p_none=0.15)


def the_moe_case():
    batch = synth.config4_batch(T=19, E=6, K=3, num_slots=3, rank=4, p_none=0.1, tag="sharding/moe")
    return synth.config4_projection(batch, "gate", d=40, n=24, tag="sharding/moe")


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    case = the_case()
    # column-parallel: no exchange until the caller gathers the columns
    y_cols, (n0, n1) = sharding.apply_column_parallel(oracle_apply, case, world, rank)
    gathered = [None] * world
    dist.all_gather_object(gathered, (y_cols, (n0, n1)))
    y_col = sharding.reassemble_columns(gathered, case.n)
    # row-parallel: the partial v are summed over the ranks

    def all_reduce_sum(v):
        t = torch.from_numpy(np.ascontiguousarray(v))
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return t.numpy()

    y_row = sharding.apply_row_parallel(oracle_shrink, oracle_expand, all_reduce_sum, case, world, rank)
    # expert-parallel MoE: every rank applies the pairs of its experts
    mcase = the_moe_case()
    local, pairs = sharding.expert_parallel_shard(mcase, world, rank)
    t = local.table
    y_local, _ = oracle.moe_lora_apply(local.ids, local.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                       local.A, local.B, local.x, local.y0)
    parts = [None] * world
    dist.all_gather_object(parts, (pairs, y_local))
    if rank == 0:
        np.save(out + ".col.npy", y_col)
        np.save(out + ".row.npy", y_row)
        y_moe = np.full((mcase.T * mcase.K, mcase.n), np.nan)
        for pr, yl in parts:
            y_moe[pr] = yl
        np.save(out + ".moe.npy", y_moe)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_ranks_reassemble_to_the_unsharded_oracle(tmp_path, world):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = str(tmp_path / "y")
    mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
    case = the_case()
    want = oracle_apply(case)
    np.testing.assert_array_equal(np.load(out + ".col.npy"), want)          # same loops on the same columns
    np.testing.assert_allclose(np.load(out + ".row.npy"), want, rtol=1e-12, atol=1e-13)   # the sum over d is regrouped
    mcase = the_moe_case()
    t = mcase.table
    want_moe, _ = oracle.moe_lora_apply(mcase.ids, mcase.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                        mcase.A, mcase.B, mcase.x, mcase.y0, x_row=mcase.x_row)
    np.testing.assert_array_equal(np.load(out + ".moe.npy"), want_moe)

"""Tensor-parallel and expert-parallel placement of the LoRA apply (host side).

The paper places LoRA tensors with the base weights they modify (section
"Scale Up": an adapter's tensors are sharded like the dense weights they
belong to; per-expert LoRA tensors are keyed by expert id and live with their
expert).  For one projection d -> n over `world` ranks that gives three cases:

* column-parallel (q, k, v, gate, up: the base weight is split on its output):
  A is replicated, B and y are split on n.  No exchange: rank k applies the
  adapter to its columns [n0, n1) of y.
* row-parallel (o, down: the base weight is split on its input): A and x are
  split on d, B is replicated.  Each rank shrinks its slice of x into a partial
  v (T x r_max, fp32); the partial v are summed over the ranks (one small
  all-reduce, T * r_max * 4 bytes) and every rank expands the sum onto its copy
  of y, which the base layer's own all-reduce has already made whole.
* expert-parallel MoE: rank k holds the experts [e0, e1); the base model's
  dispatch brings it the (token, k) pairs routed to those experts, and it
  applies their groups as a batch of its own (one pair per item).

This module holds the partition arithmetic and the order of the calls; the
arithmetic of the method stays behind the callables it is given (the CUDA
binding on a GPU, anything with the same signatures in a test).
"""
from __future__ import annotations

import dataclasses
from typing import Callable, List, Tuple

import numpy as np

from . import synth


def split_range(width: int, world: int, rank: int, multiple: int = 8) -> Tuple[int, int]:
    """Rank's share [lo, hi) of `width` columns: contiguous, multiples of `multiple`
    (bf16 vectors of 8), sizes differing by at most one multiple, the first ranks larger."""
    assert width % multiple == 0 and 0 <= rank < world
    units = width // multiple
    base, extra = divmod(units, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return lo * multiple, hi * multiple


def column_parallel_shard(case: synth.DenseCase, world: int, rank: int) -> synth.DenseCase:
    """A whole, B and y0 restricted to the rank's columns of n."""
    n0, n1 = split_range(case.n, world, rank)
    return dataclasses.replace(case, name=f"{case.name}/col{rank}of{world}", n=n1 - n0,
                               B=np.ascontiguousarray(case.B[:, :, n0:n1]),
                               y0=np.ascontiguousarray(case.y0[:, n0:n1]))


def row_parallel_shard(case: synth.DenseCase, world: int, rank: int) -> synth.DenseCase:
    """A and x restricted to the rank's columns of d; B and y0 whole."""
    d0, d1 = split_range(case.d, world, rank)
    return dataclasses.replace(case, name=f"{case.name}/row{rank}of{world}", d=d1 - d0,
                               A=np.ascontiguousarray(case.A[:, :, d0:d1]),
                               x=np.ascontiguousarray(case.x[:, d0:d1]))


def expert_parallel_shard(case: synth.MoECase, world: int, rank: int):
    """The pairs routed to the rank's experts [e0, e1) as a batch of their own:
    one item per pair (K = 1), expert ids relative to e0, the pair's adapter id,
    its x row and its row of y.  Returns (MoECase, pair indices of the full batch)."""
    e0, e1 = split_range(case.E, world, rank, multiple=1)
    flat = case.expert_ids.reshape(-1)
    pairs = np.nonzero((flat >= e0) & (flat < e1))[0]
    rows = pairs if case.x_row is None else case.x_row[pairs].astype(np.int64)
    local = synth.MoECase(
        f"{case.name}/ep{rank}of{world}", int(pairs.size), 1, e1 - e0, case.d, case.n, case.r_max, case.table,
        case.ids[pairs // case.K], (flat[pairs] - e0).astype(np.int32).reshape(-1, 1), case.pair_weight[pairs],
        None, np.ascontiguousarray(case.A[:, e0:e1]), np.ascontiguousarray(case.B[:, e0:e1]),
        np.ascontiguousarray(case.x[rows]), np.ascontiguousarray(case.y0[pairs]))
    return local, pairs


def apply_column_parallel(fused_apply: Callable, case: synth.DenseCase, world: int, rank: int):
    """fused_apply(case) -> y of the case.  Returns (y of the rank's columns, (n0, n1))."""
    return fused_apply(column_parallel_shard(case, world, rank)), split_range(case.n, world, rank)


def apply_row_parallel(shrink: Callable, expand: Callable, all_reduce_sum: Callable, case: synth.DenseCase,
                       world: int, rank: int):
    """shrink(case) -> partial v [T, r_max] (fp32 or wider) over the rank's slice of d;
    all_reduce_sum(v) -> the sum over the ranks; expand(case, v) -> y.  Returns the whole y
    (identical on every rank)."""
    shard = row_parallel_shard(case, world, rank)
    v = all_reduce_sum(shrink(shard))
    return expand(shard, v)


def reassemble_columns(parts: List[Tuple[np.ndarray, Tuple[int, int]]], n: int) -> np.ndarray:
    T = parts[0][0].shape[0]
    y = np.empty((T, n), dtype=parts[0][0].dtype)
    covered = np.zeros(n, dtype=bool)
    for yk, (n0, n1) in parts:
        assert not covered[n0:n1].any()
        y[:, n0:n1] = yk
        covered[n0:n1] = True
    assert covered.all()
    return y

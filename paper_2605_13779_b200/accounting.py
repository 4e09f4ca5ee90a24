"""Algorithmic byte and flop counts of one apply call (roofline numerators).

bytes = 2*T_active*d (x rows of tokens that have an adapter)
      + 2*sum over distinct touched adapters of rank*(d+n) (A and B once each)
      + 4*T_active*n (y read + write, bf16)
      + the id arrays.
Padding up to r_max is not counted, nor the dense T*d*n product the method
avoids.  Host-side bookkeeping for the bench and the tests only.
"""
from __future__ import annotations

import numpy as np

from .synth import DenseCase, MoECase


def algorithmic_bytes_dense(case: DenseCase) -> dict:
    """Bytes the apply must move: x rows of active tokens, each touched A and B
    once (true rank rows only), y read + write, plus ids."""
    ids = case.ids
    slots = np.where(ids >= 0, case.table.id_to_slot[np.maximum(ids, 0)], -1)
    active = slots >= 0
    t_active = int(active.sum())
    touched = np.unique(slots[active])
    sum_rank = int(case.table.slot_rank[touched].sum())
    b = {
        "x": 2 * t_active * case.d,
        "ab": 2 * sum_rank * (case.d + case.n),
        "y": 4 * t_active * case.n,
        "ids": 8 * case.T,
        "t_active": t_active,
        "distinct": int(touched.size),
        "sum_rank": sum_rank,
    }
    b["total"] = b["x"] + b["ab"] + b["y"] + b["ids"]
    b["flops"] = 2 * int(case.table.slot_rank[slots[active]].sum()) * (case.d + case.n)
    return b


def algorithmic_bytes_backward(case: DenseCase) -> dict:
    """Bytes the backward must move: x and dy rows of active tokens once, each touched A and B
    once, dx read + write (bf16), dA and dB of the touched adapters read + write (fp32, true rank
    rows), plus ids."""
    f = algorithmic_bytes_dense(case)
    b = {
        "x_dy": 2 * f["t_active"] * (case.d + case.n),
        "ab": f["ab"],
        "dx": 4 * f["t_active"] * case.d,
        "grads": 8 * f["sum_rank"] * (case.d + case.n),
        "ids": f["ids"],
    }
    b["total"] = sum(b.values())
    return b


def algorithmic_bytes_moe(case: MoECase) -> dict:
    """MoE apply: x once per distinct row read, each touched (slot, expert)
    A and B once, y read + write per active pair."""
    ids = case.ids
    slots = np.where(ids >= 0, case.table.id_to_slot[np.maximum(ids, 0)], -1)
    pair_slot = np.repeat(slots, case.K)
    pair_exp = case.expert_ids.reshape(-1).astype(np.int64)
    active = pair_slot >= 0
    p_active = int(active.sum())
    keys = np.unique(pair_exp[active] * case.table.num_slots + pair_slot[active])
    ranks = case.table.slot_rank[keys % case.table.num_slots]
    rows = np.arange(case.T * case.K) if case.x_row is None else case.x_row
    x_rows = int(np.unique(rows[active]).size)
    b = {
        "x": 2 * x_rows * case.d,
        "ab": 2 * int(ranks.sum()) * (case.d + case.n),
        "y": 4 * p_active * case.n,
        "ids": 8 * case.T + 4 * case.T * case.K,
        "p_active": p_active,
        "groups": int(keys.size),
    }
    b["total"] = b["x"] + b["ab"] + b["y"] + b["ids"]
    b["flops"] = 2 * int(case.table.slot_rank[pair_slot[active]].sum()) * (case.d + case.n)
    return b


def algorithmic_bytes_moe_backward(case: MoECase) -> dict:
    """Backward of the MoE apply: x once per distinct row read, dy once per active pair, each touched
    (slot, expert) A and B once, dx (one bf16 row per active pair) read + write, dA and dB of the touched
    blocks read + write (fp32, true ranks), plus ids."""
    f = algorithmic_bytes_moe(case)
    b = {
        "x": f["x"],
        "dy": 2 * f["p_active"] * case.n,
        "ab": f["ab"],
        "dx": 4 * f["p_active"] * case.d,
        "grads": 4 * f["ab"],            # fp32 read + write against bf16 read: 8 bytes per element against 2
        "ids": f["ids"],
    }
    b["total"] = sum(b.values())
    return b

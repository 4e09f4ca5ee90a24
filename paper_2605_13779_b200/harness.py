"""Moves synthetic cases (numpy, bf16 bit patterns) onto the device and wraps
them in the binding's handles.  Shared by the GPU tests, the smoke check and
the bench; holds no arithmetic of the method."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

from . import binding as mb
from . import synth


def upload_table(t: synth.SlotTable, device="cuda") -> mb.SlotTable:
    table = mb.SlotTable(t.catalog_size, t.num_slots, device=device)
    ids, slots, ranks, scales = t.bound()
    table.bind_many(ids, slots, ranks, scales)
    return table


@dataclass
class DeviceDense:
    case: synth.DenseCase
    table: mb.SlotTable
    pool: mb.Pool
    ids: torch.Tensor
    x: torch.Tensor
    y: torch.Tensor          # starts as y0; the apply updates it in place
    status: torch.Tensor


def upload_dense(case: synth.DenseCase, table: Optional[mb.SlotTable] = None, device="cuda") -> DeviceDense:
    if table is None:
        table = upload_table(case.table, device)
    A = mb.bf16_from_bits(case.A, device)
    B = mb.bf16_from_bits(case.B, device)
    pool = mb.Pool(A, B, case.d, case.n, case.r_max, case.table.num_slots)
    ids = torch.from_numpy(np.ascontiguousarray(case.ids, dtype=np.int64)).to(device)
    x = mb.bf16_from_bits(case.x, device)
    y = mb.bf16_from_bits(case.y0, device)
    return DeviceDense(case, table, pool, ids, x, y, mb.new_status(device))


@dataclass
class DeviceMoE:
    case: synth.MoECase
    table: mb.SlotTable
    pool: mb.Pool
    ids: torch.Tensor
    expert_ids: torch.Tensor
    x_row: Optional[torch.Tensor]
    pair_weight: torch.Tensor
    x: torch.Tensor
    y: torch.Tensor
    status: torch.Tensor


def upload_moe(case: synth.MoECase, table: Optional[mb.SlotTable] = None, device="cuda") -> DeviceMoE:
    if table is None:
        table = upload_table(case.table, device)
    A = mb.bf16_from_bits(case.A, device)
    B = mb.bf16_from_bits(case.B, device)
    pool = mb.Pool(A, B, case.d, case.n, case.r_max, case.table.num_slots, num_experts=case.E)
    ids = torch.from_numpy(np.ascontiguousarray(case.ids, dtype=np.int64)).to(device)
    expert_ids = torch.from_numpy(np.ascontiguousarray(case.expert_ids, dtype=np.int32)).to(device)
    x_row = None
    if case.x_row is not None:
        x_row = torch.from_numpy(np.ascontiguousarray(case.x_row, dtype=np.int32)).to(device)
    w = torch.from_numpy(np.ascontiguousarray(case.pair_weight, dtype=np.float32)).to(device)
    x = mb.bf16_from_bits(case.x, device)
    y = mb.bf16_from_bits(case.y0, device)
    return DeviceMoE(case, table, pool, ids, expert_ids, x_row, w, x, y, mb.new_status(device))


def y_to_f64(y: torch.Tensor) -> np.ndarray:
    """Device bf16 output widened to fp64 on the host (exact)."""
    return synth.bf16_bits_to_f64(mb.bits_from_bf16(y))

"""Shared checks of the GPU tests: tolerances of the apply and oracle calls."""
import numpy as np

from oracle import oracle
from paper_2605_13779_b200 import synth

MAX_ABS = 3e-2      # max |delta| between the bf16 GPU output and the fp64 oracle
REL_FRO = 5e-3      # relative Frobenius error over the full output


def assert_close(y_gpu: np.ndarray, y_ref: np.ndarray, what: str = ""):
    assert y_gpu.shape == y_ref.shape
    assert np.isfinite(y_gpu).all(), f"{what}: non-finite output"
    diff = np.abs(y_gpu - y_ref)
    max_abs = float(diff.max()) if diff.size else 0.0
    denom = float(np.linalg.norm(y_ref))
    rel = float(np.linalg.norm(y_gpu - y_ref)) / denom if denom > 0 else 0.0
    assert max_abs <= MAX_ABS, f"{what}: max|d|={max_abs:.4g} (max|y_ref|={np.abs(y_ref).max():.3g})"
    assert rel <= REL_FRO, f"{what}: rel-Frobenius={rel:.4g}"
    return max_abs, rel


def oracle_dense(case: synth.DenseCase, rows=None, want_v=False, y0=None):
    t = case.table
    sel = slice(None) if rows is None else rows
    y0 = case.y0 if y0 is None else y0
    return oracle.lora_apply(case.ids[sel], t.id_to_slot, t.slot_rank, t.slot_scale, case.A, case.B,
                             case.x[sel], y0[sel], want_v=want_v)


def oracle_moe(case: synth.MoECase, weighted=False, y0=None):
    t = case.table
    y0 = case.y0 if y0 is None else y0
    return oracle.moe_lora_apply(case.ids, case.expert_ids, t.id_to_slot, t.slot_rank, t.slot_scale,
                                 case.A, case.B, case.x, y0, x_row=case.x_row,
                                 pair_weight=case.pair_weight if weighted else None)

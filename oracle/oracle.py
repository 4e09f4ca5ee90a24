"""ctypes front end of the fp64 CPU oracle (lora_oracle.c).  TEST INFRASTRUCTURE.

Only the tests, the smoke check and the bench's CPU-baseline / reference legs
import this module; the CUDA product path never does.  It takes plain numpy
arrays (bf16 tensors as uint16 bit patterns) and returns fp64 results.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lora_oracle.c")
_LIB = os.path.join(_HERE, "liblora_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile lora_oracle.c with gcc (OpenMP over tokens only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_max_threads.restype = ctypes.c_int
        _lib.oracle_plan.restype = ctypes.c_int
        _lib.oracle_lora_apply.restype = ctypes.c_int32
        _lib.oracle_moe_lora_apply.restype = ctypes.c_int32
    return _lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def plan(ids, id_to_slot, num_slots: int, expert_ids=None, num_experts: int = 0) -> dict:
    """Canonical segment plan: items ordered by key then index; one segment per
    distinct key.  Dense key = slot; MoE key = expert * num_slots + slot."""
    lib = _load()
    ids = _c(ids, np.int64)
    id_to_slot = _c(id_to_slot, np.int32)
    T = ids.shape[0]
    if expert_ids is not None:
        expert_ids = _c(expert_ids, np.int32)
        K = expert_ids.size // max(T, 1) if T else 1
        K = max(K, 1)
        expert_flat = expert_ids.reshape(-1)
    else:
        K, expert_flat = 1, None
    P = T * K
    perm = np.zeros(P, dtype=np.int32)
    seg_key = np.zeros(P, dtype=np.int32)
    seg_start = np.zeros(P + 1, dtype=np.int32)
    S = ctypes.c_int32(0)
    n_active = ctypes.c_int32(0)
    missing = ctypes.c_int32(0)
    bad_expert = ctypes.c_int32(0)
    lib.oracle_plan(_p(ids), ctypes.c_int32(T), _p(expert_flat), ctypes.c_int32(K),
                    ctypes.c_int32(num_experts), _p(id_to_slot), ctypes.c_int64(id_to_slot.shape[0]),
                    ctypes.c_int32(num_slots), _p(perm), _p(seg_key), _p(seg_start),
                    ctypes.byref(S), ctypes.byref(n_active), ctypes.byref(missing),
                    ctypes.byref(bad_expert))
    S, m = S.value, n_active.value
    return {
        "perm": perm[:m].copy(),
        "seg_key": seg_key[:S].copy(),
        "seg_start": seg_start[:S + 1].copy(),
        "S": S,
        "n_active": m,
        "n_not_resident": missing.value,
        "n_bad_expert": bad_expert.value,
    }


def lora_apply(ids, id_to_slot, slot_rank, slot_scale, A, B, x, y0, *, a_layout: str = "rd",
               num_threads: int = 0, want_v: bool = False):
    """Dense apply.  A is [slots, r_max, d] for a_layout "rd" or
    [slots, d, r_max] for "dr"; B is [slots, r_max, n]; x [T, d]; y0 [T, n]
    (all bf16 bit patterns).  Returns (y_ref fp64 [T, n], v fp64 [T, r_max] or
    None, number of tokens whose id was not resident)."""
    lib = _load()
    ids = _c(ids, np.int64)
    id_to_slot = _c(id_to_slot, np.int32)
    slot_rank = _c(slot_rank, np.int32)
    slot_scale = _c(slot_scale, np.float32)
    A = _c(A, np.uint16)
    B = _c(B, np.uint16)
    x = _c(x, np.uint16)
    y0 = _c(y0, np.uint16)
    T = ids.shape[0]
    num_slots = slot_rank.shape[0]
    n = B.shape[2]
    r_max = B.shape[1]
    if a_layout == "rd":
        assert A.shape[1] == r_max
        d = A.shape[2]
        a_strides = (r_max * d, 1, d)           # slot, i (input feature), j (rank)
    elif a_layout == "dr":
        assert A.shape[2] == r_max
        d = A.shape[1]
        a_strides = (r_max * d, r_max, 1)
    else:
        raise ValueError(a_layout)
    assert x.shape == (T, d) and y0.shape == (T, n)
    y_ref = np.empty((T, n), dtype=np.float64)
    v = np.empty((T, r_max), dtype=np.float64) if want_v else None
    missing = lib.oracle_lora_apply(
        ctypes.c_int32(T), ctypes.c_int32(d), ctypes.c_int32(n), ctypes.c_int32(r_max),
        _p(ids), _p(id_to_slot), ctypes.c_int64(id_to_slot.shape[0]), ctypes.c_int32(num_slots),
        _p(slot_rank), _p(slot_scale),
        _p(A), ctypes.c_int64(a_strides[0]), ctypes.c_int64(a_strides[1]), ctypes.c_int64(a_strides[2]),
        _p(B), ctypes.c_int64(r_max * n), ctypes.c_int64(n), ctypes.c_int64(1),
        _p(x), ctypes.c_int64(d), _p(y0), ctypes.c_int64(n),
        _p(y_ref), _p(v), ctypes.c_int32(num_threads))
    return y_ref, v, int(missing)


def moe_lora_apply(ids, expert_ids, id_to_slot, slot_rank, slot_scale, A, B, x, y0, *,
                   x_row=None, pair_weight=None, num_threads: int = 0):
    """MoE expert LoRA apply.  A is [slots, E, d, r_max], B is
    [slots, E, r_max, n], expert_ids [T, K], y0 [T*K, n].  Returns
    (Y_ref fp64 [T*K, n], number of tokens whose id was not resident)."""
    lib = _load()
    ids = _c(ids, np.int64)
    expert_ids = _c(expert_ids, np.int32)
    id_to_slot = _c(id_to_slot, np.int32)
    slot_rank = _c(slot_rank, np.int32)
    slot_scale = _c(slot_scale, np.float32)
    A = _c(A, np.uint16)
    B = _c(B, np.uint16)
    x = _c(x, np.uint16)
    y0 = _c(y0, np.uint16)
    T = ids.shape[0]
    K = expert_ids.shape[1] if expert_ids.ndim == 2 else 1
    num_slots, E, d, r_max = A.shape
    n = B.shape[3]
    assert B.shape == (num_slots, E, r_max, n)
    P = T * K
    assert y0.shape == (P, n) and x.shape[1] == d
    if x_row is not None:
        x_row = _c(x_row, np.int32)
        assert x_row.shape == (P,)
    else:
        assert x.shape[0] >= P
    if pair_weight is not None:
        pair_weight = _c(pair_weight, np.float32)
        assert pair_weight.shape == (P,)
    y_ref = np.empty((P, n), dtype=np.float64)
    missing = lib.oracle_moe_lora_apply(
        ctypes.c_int32(T), ctypes.c_int32(K), ctypes.c_int32(E), ctypes.c_int32(d), ctypes.c_int32(n),
        _p(ids), _p(expert_ids.reshape(-1)), _p(id_to_slot), ctypes.c_int64(id_to_slot.shape[0]),
        ctypes.c_int32(num_slots), _p(slot_rank), _p(slot_scale),
        _p(A), ctypes.c_int64(E * d * r_max), ctypes.c_int64(d * r_max), ctypes.c_int64(r_max),
        ctypes.c_int64(1),
        _p(B), ctypes.c_int64(E * r_max * n), ctypes.c_int64(r_max * n), ctypes.c_int64(n),
        ctypes.c_int64(1),
        _p(x), ctypes.c_int64(d), _p(x_row), _p(pair_weight),
        _p(y0), ctypes.c_int64(n), _p(y_ref), ctypes.c_int32(num_threads))
    return y_ref, int(missing)


def moe_lora_apply_combine(ids, expert_ids, id_to_slot, slot_rank, slot_scale, A, B, x, y0_tokens, pair_weight, *,
                           x_row=None, num_threads: int = 0):
    """Router-weighted combine of the MoE expert LoRA update into the token's row
    (paper, "Scale Up": per-expert LoRA tensors keyed by expert id; the routed
    experts' outputs of a token are combined with the router's weights):

        Y[t, :] = Y0[t, :] + sum over k of  w[t, k] * s * (X[row(t, k), :] . A[sigma][e]) . B[sigma][e]

    Written as the per-pair oracle on a zero start (each pair's weighted update
    in fp64) followed by the plain sum over k, in k order.  y0_tokens is bf16
    bits [T, n]; returns (Y_ref fp64 [T, n], tokens whose id was not resident)."""
    ids = _c(ids, np.int64)
    expert_ids = _c(expert_ids, np.int32)
    T = ids.shape[0]
    K = expert_ids.shape[1] if expert_ids.ndim == 2 else 1
    n = np.asarray(B).shape[3]
    y0_tokens = _c(y0_tokens, np.uint16)
    assert y0_tokens.shape == (T, n)
    zero = np.zeros((T * K, n), dtype=np.uint16)
    per_pair, missing = moe_lora_apply(ids, expert_ids, id_to_slot, slot_rank, slot_scale, A, B, x, zero,
                                       x_row=x_row, pair_weight=pair_weight, num_threads=num_threads)
    y_ref = (y0_tokens.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    for k in range(K):
        y_ref = y_ref + per_pair[k::K]
    return y_ref, missing

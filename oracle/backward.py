"""fp64 CPU oracle of the LoRA backward over padded slots.  TEST INFRASTRUCTURE.

Only the tests, the smoke check and the bench's CPU-baseline leg import this
module; the CUDA product path never does.

The paper trains adapters in time slices over a shared frozen base (section
"Time-Sliced Multi-LoRA Training": workers are configured for adapter-shape
limits, adapters of smaller rank are padded to the slot's shape and masked, and
kernels that update several adapters in one batch are named as the
alternative).  It prints no formula for the backward; what is computed here is the plain derivative of the
update the forward path applies,

    y[t, :] = y0[t, :] + s * (x[t, :] . A^T) . B        A: [rank, d], B: [rank, n] of the token's slot,

with respect to x, A and B, for an upstream gradient dy = dL/dy:

    u[t, :]  = dy[t, :] . B^T                      (rank)
    v[t, :]  = x[t, :] . A^T                       (rank)
    dx[t, :] = dx0[t, :] + s * u[t, :] . A         (d)
    dA[slot][k, :] = dA0 + s * sum over the slot's tokens of  u[t, k] * x[t, :]
    dB[slot][k, :] = dB0 + s * sum over the slot's tokens of  v[t, k] * dy[t, :]

Rows k >= rank of a slot (the padding) and slots without tokens keep dA0 / dB0;
tokens without an adapter (id -1) or whose id is not resident contribute
nothing and keep their dx0 row.  Token by token, nothing rounded, no blocking.
Pinned in tests/test_oracle_backward.py (central differences of the forward
oracle, two-matmul closed form, masks, a hand-worked example): parity pinned.
"""
from __future__ import annotations

from typing import Optional, Tuple

import numpy as np


def _bf16(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp64, exact."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def lora_backward(ids, id_to_slot, slot_rank, slot_scale, A, B, x, dy, *, dx0: Optional[np.ndarray] = None,
                  dA0: Optional[np.ndarray] = None, dB0: Optional[np.ndarray] = None
                  ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, int]:
    """A [slots, r_max, d], B [slots, r_max, n], x [T, d], dy [T, n]: bf16 bit patterns.
    dx0 (bf16 bits [T, d]) and dA0 / dB0 (fp64 or fp32 arrays shaped like A / B) are the
    starting values; zero when omitted.  Returns (dx [T, d], dA, dB, tokens whose id was not
    resident), all fp64."""
    ids = np.asarray(ids, dtype=np.int64)
    id_to_slot = np.asarray(id_to_slot, dtype=np.int32)
    slot_rank = np.asarray(slot_rank, dtype=np.int32)
    slot_scale = np.asarray(slot_scale, dtype=np.float32)
    Af, Bf, xf, gf = _bf16(A), _bf16(B), _bf16(x), _bf16(dy)
    T, d = xf.shape
    n = gf.shape[1]
    assert Af.shape[0] == Bf.shape[0] == slot_rank.shape[0] and Af.shape[2] == d and Bf.shape[2] == n
    dx = np.zeros((T, d)) if dx0 is None else _bf16(dx0)
    dA = np.zeros(Af.shape) if dA0 is None else np.array(dA0, dtype=np.float64)
    dB = np.zeros(Bf.shape) if dB0 is None else np.array(dB0, dtype=np.float64)
    missing = 0
    for t in range(T):
        cid = int(ids[t])
        if cid == -1:
            continue
        slot = int(id_to_slot[cid]) if 0 <= cid < id_to_slot.shape[0] else -1
        if slot < 0 or slot >= slot_rank.shape[0]:
            missing += 1
            continue
        r = int(slot_rank[slot])
        s = float(slot_scale[slot])
        a = Af[slot, :r, :]          # [r, d]
        b = Bf[slot, :r, :]          # [r, n]
        u = b @ gf[t]                # dy . B^T
        v = a @ xf[t]                # x . A^T
        dx[t] += s * (u @ a)
        dA[slot, :r, :] += s * np.outer(u, xf[t])
        dB[slot, :r, :] += s * np.outer(v, gf[t])
    return dx, dA, dB, missing


def moe_lora_backward(ids, expert_ids, id_to_slot, slot_rank, slot_scale, A, B, x, dy, *, x_row=None,
                      pair_weight=None, dx0: Optional[np.ndarray] = None, dA0: Optional[np.ndarray] = None,
                      dB0: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray, np.ndarray, int]:
    """The same derivative for per-expert LoRA tensors keyed by expert id (section "Scale Up"; packed
    layout of the packed-loader table): pair p = (token t, k-th routed expert e) of a token whose
    adapter sits in slot sigma was updated by

        y[p, :] = y0[p, :] + w_p * s * (x[row_p, :] . A[sigma, e]) . B[sigma, e]     A: [d, r], B: [r, n],

    and for an upstream gradient dy [T*K, n] (one row per pair)

        u = B[sigma, e] . dy[p],   v = x[row_p] . A[sigma, e]                         (rank values)
        dx[p, :]          = dx0[p, :] + w_p * s * A[sigma, e] . u       one row per PAIR: the rows of the
                                                                         pairs that read one x row are the caller's to add
        dA[sigma, e][:, k] += w_p * s * u[k] * x[row_p, :]
        dB[sigma, e][k, :] += w_p * s * v[k] * dy[p, :]

    Ranks k >= rank of the slot, (slot, expert) blocks without pairs, pairs of tokens without an
    adapter, of ids that are not resident and of expert ids outside [0, E) change nothing; the routing
    weights are constants (no derivative with respect to them).  A is [slots, E, d, r_max], B is
    [slots, E, r_max, n], x [rows, d], dy [T*K, n]: bf16 bit patterns; dx0 bf16 bits [T*K, d]; dA0 / dB0
    fp32 or fp64 shaped like A / B.  Returns (dx [T*K, d], dA, dB, tokens whose id was not resident), fp64.
    Pair by pair, nothing rounded.  Pinned in tests/test_oracle_backward.py: parity pinned."""
    ids = np.asarray(ids, dtype=np.int64)
    expert_ids = np.asarray(expert_ids, dtype=np.int32)
    id_to_slot = np.asarray(id_to_slot, dtype=np.int32)
    slot_rank = np.asarray(slot_rank, dtype=np.int32)
    slot_scale = np.asarray(slot_scale, dtype=np.float32)
    Af, Bf, xf, gf = _bf16(A), _bf16(B), _bf16(x), _bf16(dy)
    T = ids.shape[0]
    K = expert_ids.shape[1] if expert_ids.ndim == 2 else 1
    experts = expert_ids.reshape(T, K)
    num_slots, E, d, r_max = Af.shape
    n = Bf.shape[3]
    P = T * K
    assert Bf.shape == (num_slots, E, r_max, n) and gf.shape == (P, n) and xf.shape[1] == d
    rows = np.arange(P) if x_row is None else np.asarray(x_row, dtype=np.int64)
    w = np.ones(P) if pair_weight is None else np.asarray(pair_weight, dtype=np.float32).astype(np.float64)
    dx = np.zeros((P, d)) if dx0 is None else _bf16(dx0)
    dA = np.zeros(Af.shape) if dA0 is None else np.array(dA0, dtype=np.float64)
    dB = np.zeros(Bf.shape) if dB0 is None else np.array(dB0, dtype=np.float64)
    missing = 0
    for t in range(T):
        cid = int(ids[t])
        if cid == -1:
            continue
        slot = int(id_to_slot[cid]) if 0 <= cid < id_to_slot.shape[0] else -1
        if slot < 0 or slot >= num_slots:
            missing += 1
            continue
        r = int(slot_rank[slot])
        s = float(slot_scale[slot])
        for k in range(K):
            e = int(experts[t, k])
            if e < 0 or e >= E:
                continue
            p = t * K + k
            a = Af[slot, e, :, :r]       # [d, r]
            b = Bf[slot, e, :r, :]       # [r, n]
            xr = xf[rows[p]]
            u = b @ gf[p]
            v = xr @ a
            c = w[p] * s
            dx[p] += c * (a @ u)
            dA[slot, e, :, :r] += c * np.outer(xr, u)
            dB[slot, e, :r, :] += c * np.outer(v, gf[p])
    return dx, dA, dB, missing

"""Seeded synthetic workloads for the mixed-adapter LoRA apply.

This module only *draws inputs*: adapter ids, slot tables, router choices and
bf16 tensors with the shapes, value distributions and structure of the five
benchmark settings (4B-dense decode layer, 32B-dense segmented prefill,
30B-A3B MoE expert LoRA, million-entry catalog slice, and a tiny single
projection).  It holds none of the method's arithmetic: no shrink, no expand,
no segment planning.  Both the CUDA path and the CPU oracle are handed the
buffers produced here; neither is imported from here.

Everything is numpy on the host.  bf16 tensors are carried as uint16 bit
patterns so that the two consumers see identical bits.

Workload structure follows the paper's serving description: one resident base,
a bounded set of GPU slots (at most 64 distinct adapters in a decoding batch,
"Scale Out: Policy-Population Serving", cache-tier table), slots allocated at a
configured maximum rank with smaller adapters padded ("Time-Sliced Multi-LoRA
Training"), per-expert MoE LoRA tensors stacked along an expert axis (packed
representation, "Policy-Population Serving" evaluation), and a catalog of up
to 10^6 ids of which only a bounded subset is resident.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field
from typing import Dict, Optional, Tuple

import numpy as np

BASE_SEED = 20260513
BF16_NAN_BITS = 0x7FC0

# The seven LoRA target projections of the 4B-dense decode layer (d -> n).
QWEN3_4B_PROJECTIONS: Dict[str, Tuple[int, int]] = {
    "q": (2560, 4096),
    "k": (2560, 1024),
    "v": (2560, 1024),
    "o": (4096, 2560),
    "gate": (2560, 9728),
    "up": (2560, 9728),
    "down": (9728, 2560),
}
QWEN3_4B_LAYERS = 36

# 32B-dense segmented prefill projections.
DENSE_32B_PROJECTIONS: Dict[str, Tuple[int, int]] = {
    "attn": (5120, 5120),
    "up": (5120, 25600),
    "down": (25600, 5120),
}

# 30B-A3B MoE expert FFN (hidden 2048, expert width 768).
MOE_30B_PROJECTIONS: Dict[str, Tuple[int, int]] = {
    "gate": (2048, 768),
    "up": (2048, 768),
    "down": (768, 2048),
}
MOE_30B_LAYERS = 48


# --------------------------------------------------------------------------
# random streams and bf16 bit handling
# --------------------------------------------------------------------------
def stream(*names) -> np.random.Generator:
    """Counter-based generator keyed by (BASE_SEED, names...).  The key is a
    blake2b digest, so it does not depend on Python's per-process hash salt."""
    text = "/".join(str(x) for x in (BASE_SEED,) + tuple(names))
    digest = hashlib.blake2b(text.encode(), digest_size=16).digest()
    key = np.frombuffer(digest, dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round to nearest, ties to even); uint16 bits."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        out[nan] = BF16_NAN_BITS
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to float32 (exact)."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


def normal_bf16(rng: np.random.Generator, shape, std: float, chunk: int = 1 << 24) -> np.ndarray:
    """N(0, std^2) drawn in fp32, rounded to bf16 bits.  Drawn in chunks so the
    fp32 temporary stays small for the prefill-sized tensors."""
    total = int(np.prod(shape))
    out = np.empty(total, dtype=np.uint16)
    pos = 0
    while pos < total:
        m = min(chunk, total - pos)
        v = rng.standard_normal(m, dtype=np.float32)
        if std != 1.0:
            v *= np.float32(std)
        out[pos:pos + m] = f32_to_bf16_bits(v)
        pos += m
    return out.reshape(shape)


def bounded_zipf(rng: np.random.Generator, n_items: int, s: float, size: int) -> np.ndarray:
    """Popularity ranks 0..n_items-1 with P(rank k) proportional to (k+1)^-s,
    by inverse CDF on an fp64 cumulative table."""
    w = np.arange(1, n_items + 1, dtype=np.float64) ** (-float(s))
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = rng.random(size)
    k = np.searchsorted(cdf, u, side="right")
    return np.minimum(k, n_items - 1).astype(np.int64)


# --------------------------------------------------------------------------
# case containers
# --------------------------------------------------------------------------
@dataclass
class SlotTable:
    """Catalog id -> GPU slot, and per-slot true rank and scale."""
    catalog_size: int
    num_slots: int
    id_to_slot: np.ndarray   # int32 [catalog_size]; -1 = not resident
    slot_rank: np.ndarray    # int32 [num_slots]; 0 = empty slot
    slot_scale: np.ndarray   # float32 [num_slots]

    def bound(self):
        """(catalog id, slot, rank, scale) for every resident id, in id order."""
        ids = np.nonzero(self.id_to_slot >= 0)[0].astype(np.int64)
        slots = self.id_to_slot[ids]
        return ids, slots, self.slot_rank[slots], self.slot_scale[slots]


@dataclass
class DenseCase:
    name: str
    T: int
    d: int
    n: int
    r_max: int
    table: SlotTable
    ids: np.ndarray          # int64 [T]; -1 = no adapter
    A: np.ndarray            # uint16 [num_slots, r_max, d]   (rank-major, d contiguous)
    B: np.ndarray            # uint16 [num_slots, r_max, n]
    x: np.ndarray            # uint16 [T, d]
    y0: np.ndarray           # uint16 [T, n]
    meta: dict = field(default_factory=dict)


@dataclass
class MoECase:
    name: str
    T: int
    K: int
    E: int
    d: int
    n: int
    r_max: int
    table: SlotTable
    ids: np.ndarray          # int64 [T]
    expert_ids: np.ndarray   # int32 [T, K]
    pair_weight: np.ndarray  # float32 [T*K] (softmax over the K selected logits)
    x_row: Optional[np.ndarray]  # int32 [T*K] row of x read by pair p, or None = identity
    A: np.ndarray            # uint16 [num_slots, E, d, r_max]  (packed: expert axis stacked)
    B: np.ndarray            # uint16 [num_slots, E, r_max, n]
    x: np.ndarray            # uint16 [rows, d]
    y0: np.ndarray           # uint16 [T*K, n]
    meta: dict = field(default_factory=dict)


def identity_table(num_slots: int, ranks, scale: float = 2.0) -> SlotTable:
    """Catalog of num_slots ids, id i resident in slot i."""
    ranks = np.asarray(ranks, dtype=np.int32)
    assert ranks.shape == (num_slots,)
    return SlotTable(
        catalog_size=num_slots,
        num_slots=num_slots,
        id_to_slot=np.arange(num_slots, dtype=np.int32),
        slot_rank=ranks.copy(),
        slot_scale=np.full(num_slots, scale, dtype=np.float32),
    )


def dense_pool(rng, table: SlotTable, r_max: int, d: int, n: int, std: float = 0.02,
               pad_bits: int = BF16_NAN_BITS):
    """A[slot][r_max][d], B[slot][r_max][n]; rows at or beyond a slot's true
    rank (and all rows of empty slots) hold pad_bits: padding that a correct
    apply never reads."""
    S = table.num_slots
    A = normal_bf16(rng, (S, r_max, d), std)
    B = normal_bf16(rng, (S, r_max, n), std)
    row = np.arange(r_max)[None, :]
    pad = row >= table.slot_rank[:, None]
    A[pad] = pad_bits
    B[pad] = pad_bits
    return A, B


def moe_pool(rng, table: SlotTable, E: int, r_max: int, d: int, n: int, std: float = 0.02,
             pad_bits: int = BF16_NAN_BITS):
    """A[slot][E][d][r_max], B[slot][E][r_max][n] with padded rank columns/rows
    set to pad_bits."""
    S = table.num_slots
    A = normal_bf16(rng, (S, E, d, r_max), std)
    B = normal_bf16(rng, (S, E, r_max, n), std)
    col = np.arange(r_max)
    for s in range(S):
        padc = col >= table.slot_rank[s]
        if padc.any():
            A[s][:, :, padc] = pad_bits
            B[s][:, padc, :] = pad_bits
    return A, B


# --------------------------------------------------------------------------
# generic small cases (tests sweep these)
# --------------------------------------------------------------------------
def random_dense_case(name: str, T: int, d: int, n: int, num_slots: int, ranks, r_max: int,
                      p_none: float = 0.1, scale: float = 2.0, zipf_s: Optional[float] = None,
                      std: float = 0.02) -> DenseCase:
    rng = stream(name, "ids")
    table = identity_table(num_slots, ranks, scale)
    if T == 0:
        ids = np.zeros(0, dtype=np.int64)
    elif zipf_s is None:
        ids = rng.integers(0, num_slots, size=T).astype(np.int64)
    else:
        pop = bounded_zipf(rng, num_slots, zipf_s, T)
        ids = stream(name, "perm").permutation(num_slots)[pop].astype(np.int64)
    if p_none > 0 and T > 0:
        ids[rng.random(T) < p_none] = -1
    A, B = dense_pool(stream(name, "pool"), table, r_max, d, n, std)
    x = normal_bf16(stream(name, "x"), (T, d), 1.0)
    y0 = normal_bf16(stream(name, "y0"), (T, n), 1.0)
    return DenseCase(name, T, d, n, r_max, table, ids, A, B, x, y0)


def config1() -> DenseCase:
    """Single projection 2560 -> 2560, T=64, four rank-8 adapters, scale 2,
    id uniform over {0..3} with probability 0.1 of 'no adapter'."""
    return random_dense_case("config1", T=64, d=2560, n=2560, num_slots=4,
                             ranks=[8, 8, 8, 8], r_max=8, p_none=0.1)


# --------------------------------------------------------------------------
# config 2: 4B-dense decode layer
# --------------------------------------------------------------------------
@dataclass
class DecodeBatch:
    T: int
    table: SlotTable
    ids: np.ndarray
    r_max: int


def config2_batch(T: int = 256, num_slots: int = 64, zipf_s: float = 1.1,
                  rank_choices=(1, 8, 16, 32), tag: str = "config2") -> DecodeBatch:
    """One decode step: T requests, one token each; request -> adapter bounded
    Zipf(1.1) over 64 resident adapters through a seeded permutation; rank per
    adapter iid uniform over {1, 8, 16, 32}; every request has an adapter."""
    rng = stream(tag, "batch")
    ranks = rng.choice(np.asarray(rank_choices, dtype=np.int32), size=num_slots)
    table = identity_table(num_slots, ranks, 2.0)
    pop = bounded_zipf(rng, num_slots, zipf_s, T)
    ids = stream(tag, "perm").permutation(num_slots)[pop].astype(np.int64)
    return DecodeBatch(T, table, ids, int(max(rank_choices)))


def config2_projection(batch: DecodeBatch, proj: str, layer: int = 0, tag: str = "config2") -> DenseCase:
    d, n = QWEN3_4B_PROJECTIONS[proj]
    A, B = dense_pool(stream(tag, proj, layer, "pool"), batch.table, batch.r_max, d, n)
    x = normal_bf16(stream(tag, proj, layer, "x"), (batch.T, d), 1.0)
    y0 = normal_bf16(stream(tag, proj, layer, "y0"), (batch.T, n), 1.0)
    return DenseCase(f"{tag}/{proj}/L{layer}", batch.T, d, n, batch.r_max, batch.table,
                     batch.ids, A, B, x, y0, meta={"proj": proj, "layer": layer})


# --------------------------------------------------------------------------
# config 3: segmented prefill on 32B-dense shapes
# --------------------------------------------------------------------------
@dataclass
class PrefillBatch:
    T: int
    table: SlotTable
    ids: np.ndarray
    r_max: int
    lengths: np.ndarray
    request_adapter: np.ndarray


def config3_batch(num_requests: int = 32, len_lo: int = 128, len_hi: int = 1024, rank: int = 64,
                  bijection: bool = True, tag: str = "config3") -> PrefillBatch:
    """32 requests with lengths uniform in [128, 1024]; each request's tokens
    are contiguous and carry the request's adapter.  bijection=True binds
    request i to a distinct adapter (seeded permutation); bijection=False draws
    adapters iid, so one adapter can own several non-adjacent requests."""
    rng = stream(tag, "batch", bijection)
    lengths = rng.integers(len_lo, len_hi + 1, size=num_requests).astype(np.int64)
    if bijection:
        req_adapter = rng.permutation(num_requests).astype(np.int64)
    else:
        req_adapter = rng.integers(0, num_requests, size=num_requests).astype(np.int64)
    ids = np.repeat(req_adapter, lengths)
    table = identity_table(num_requests, np.full(num_requests, rank, dtype=np.int32), 2.0)
    return PrefillBatch(int(lengths.sum()), table, ids, rank, lengths, req_adapter)


def config3_projection(batch: PrefillBatch, d: int, n: int, tag: str = "config3") -> DenseCase:
    A, B = dense_pool(stream(tag, d, n, "pool"), batch.table, batch.r_max, d, n)
    x = normal_bf16(stream(tag, d, n, "x"), (batch.T, d), 1.0)
    y0 = normal_bf16(stream(tag, d, n, "y0"), (batch.T, n), 1.0)
    return DenseCase(f"{tag}/{d}x{n}", batch.T, d, n, batch.r_max, batch.table, batch.ids,
                     A, B, x, y0)


# --------------------------------------------------------------------------
# config 4: 30B-A3B-shaped MoE expert LoRA
# --------------------------------------------------------------------------
def topk_route(logits: np.ndarray, K: int):
    """Top-K experts per token: larger logit first, lower expert index on
    ties; weights are the softmax over the K selected logits."""
    order = np.argsort(-logits, axis=1, kind="stable")[:, :K]
    sel = np.take_along_axis(logits, order, axis=1).astype(np.float64)
    sel -= sel.max(axis=1, keepdims=True)
    w = np.exp(sel)
    w /= w.sum(axis=1, keepdims=True)
    return order.astype(np.int32), w.astype(np.float32)


@dataclass
class MoEBatch:
    T: int
    K: int
    E: int
    table: SlotTable
    ids: np.ndarray
    expert_ids: np.ndarray
    pair_weight: np.ndarray
    r_max: int


def config4_batch(T: int = 4096, E: int = 128, K: int = 8, num_slots: int = 16, rank: int = 16,
                  contiguous_requests: bool = False, p_none: float = 0.0,
                  tag: str = "config4") -> MoEBatch:
    """Router logits fp32 N(0,1) [T, E], top-K routing, adapter per token iid
    uniform over the resident adapters (or, with contiguous_requests, 32 equal
    contiguous requests each bound to one adapter)."""
    rng = stream(tag, "batch", T, E, K, num_slots, contiguous_requests)
    logits = rng.standard_normal((T, E), dtype=np.float32)
    expert_ids, w = topk_route(logits, K)
    if contiguous_requests:
        nreq = min(32, max(T, 1))
        req_adapter = rng.integers(0, num_slots, size=nreq)
        ids = req_adapter[(np.arange(T) * nreq) // max(T, 1)].astype(np.int64)
    else:
        ids = rng.integers(0, num_slots, size=T).astype(np.int64)
    if p_none > 0:
        ids[rng.random(T) < p_none] = -1
    table = identity_table(num_slots, np.full(num_slots, rank, dtype=np.int32), 2.0)
    return MoEBatch(T, K, E, table, ids, expert_ids, w.reshape(-1), rank)


def config4_projection(batch: MoEBatch, proj: str, d: Optional[int] = None, n: Optional[int] = None,
                       layer: int = 0, tag: str = "config4") -> MoECase:
    """gate/up read the token's hidden row (x_row[p] = p // K), the same hidden
    states for both; down reads the per-pair intermediate row (identity)."""
    if d is None or n is None:
        d, n = MOE_30B_PROJECTIONS[proj]
    P = batch.T * batch.K
    A, B = moe_pool(stream(tag, proj, layer, d, n, "pool"), batch.table, batch.E, batch.r_max, d, n)
    if proj == "down":
        x = normal_bf16(stream(tag, proj, layer, "x"), (P, d), 1.0)
        x_row = None
    else:
        x = normal_bf16(stream(tag, "gate", layer, "x"), (batch.T, d), 1.0)
        x_row = (np.arange(P, dtype=np.int64) // batch.K).astype(np.int32)
    y0 = normal_bf16(stream(tag, proj, layer, "y0"), (P, n), 1.0)
    return MoECase(f"{tag}/{proj}/L{layer}", batch.T, batch.K, batch.E, d, n, batch.r_max,
                   batch.table, batch.ids, batch.expert_ids, batch.pair_weight, x_row, A, B, x, y0,
                   meta={"proj": proj})


# --------------------------------------------------------------------------
# config 5: million-adapter catalog slice
# --------------------------------------------------------------------------
def config5(T: int = 2048, catalog_size: int = 1_000_000, num_slots: int = 4096,
            d: int = 7168, n: int = 7168, zipf_s: float = 0.9, leave_unbound: int = 0,
            tag: str = "config5") -> DenseCase:
    """10^6 rank-1 catalog ids, 4096 resident slots.  The batch is drawn
    first (Zipf(0.9) over the catalog through a seeded permutation); every
    distinct id in it is bound to a slot in seeded random slot order, and the
    remaining slots are filled with the most popular ids not yet resident.
    leave_unbound > 0 unbinds that many batch ids again (contract-violation
    tests: such tokens must be reported and left untouched)."""
    rng = stream(tag, "batch", T, catalog_size, num_slots)
    pop = bounded_zipf(rng, catalog_size, zipf_s, T)
    pop_to_id = stream(tag, "perm", catalog_size).permutation(catalog_size).astype(np.int64)
    ids = pop_to_id[pop]
    distinct = np.unique(ids)
    assert distinct.size <= num_slots
    slot_order = rng.permutation(num_slots).astype(np.int32)
    id_to_slot = np.full(catalog_size, -1, dtype=np.int32)
    id_to_slot[distinct] = slot_order[:distinct.size]
    filled = distinct.size
    k = 0
    while filled < num_slots and k < catalog_size:
        cid = pop_to_id[k]
        if id_to_slot[cid] < 0:
            id_to_slot[cid] = slot_order[filled]
            filled += 1
        k += 1
    unbound = np.zeros(0, dtype=np.int64)
    if leave_unbound > 0:
        unbound = rng.choice(distinct, size=min(leave_unbound, distinct.size), replace=False)
        id_to_slot[unbound] = -1
    slot_rank = np.zeros(num_slots, dtype=np.int32)
    slot_rank[id_to_slot[id_to_slot >= 0]] = 1
    table = SlotTable(catalog_size, num_slots, id_to_slot, slot_rank,
                      np.full(num_slots, 2.0, dtype=np.float32))
    A, B = dense_pool(stream(tag, "pool", d, n), table, 1, d, n)
    x = normal_bf16(stream(tag, "x", d), (T, d), 1.0)
    y0 = normal_bf16(stream(tag, "y0", n), (T, n), 1.0)
    return DenseCase(tag, T, d, n, 1, table, ids, A, B, x, y0,
                     meta={"distinct": int(distinct.size), "unbound": unbound})


# --------------------------------------------------------------------------
# adapter-file shape accounting (sanity pins for the generators' shapes)
# --------------------------------------------------------------------------
def dense_adapter_params(rank: int, projections=QWEN3_4B_PROJECTIONS, layers: int = QWEN3_4B_LAYERS) -> int:
    """Number of LoRA parameters of a dense adapter: rank * (d + n) per target
    projection per layer."""
    return layers * rank * sum(d + n for d, n in projections.values())


def moe_adapter_tensor_counts(layers: int = MOE_30B_LAYERS, experts: int = 128, hidden: int = 2048,
                              ffn: int = 768, q_out: int = 4096, kv_out: int = 512, rank: int = 1):
    """Tensor and byte counts of a per-expert MoE adapter (attention q,k,v,o
    plus per-expert gate/up/down) before and after stacking the per-expert
    tensors of one projection of one layer along an expert axis."""
    expert_tensors = layers * experts * 3 * 2
    attn_tensors = layers * 4 * 2
    packed_groups = layers * 3 * 2
    per_expert_elems = rank * ((hidden + ffn) * 2 + (ffn + hidden))
    attn_elems = rank * ((hidden + q_out) + 2 * (hidden + kv_out) + (q_out + hidden))
    total_bytes = layers * (experts * per_expert_elems + attn_elems) * 2
    # tensors of at most 4 KB at bf16: every expert tensor, and the attention
    # tensors whose long side is at most 2048 elements.
    attn_dims = [hidden, q_out, hidden, kv_out, hidden, kv_out, q_out, hidden]
    small_attn = sum(1 for v in attn_dims if v * rank * 2 <= 4096)
    return {
        "tensors": expert_tensors + attn_tensors,
        "packed_tensors": packed_groups + attn_tensors,
        "packed_groups": packed_groups,
        "copied": attn_tensors,
        "small_tensors": expert_tensors + layers * small_attn,
        "bytes": total_bytes,
    }

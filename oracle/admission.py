"""CPU oracle of the admission step that precedes the apply.  TEST INFRASTRUCTURE.

Only the tests import this module; the CUDA product path never does, and it
shares no code with it.  Plain Python / numpy loops, written from the paper's
description:

* Admission from the packed representation.  An exported MoE LoRA adapter is a
  moderate number of bytes in tens of thousands of tiny per-expert tensors; the
  paper's packed serving representation stacks the per-expert tensors of a
  projection along an expert axis (section "Policy-Population Multi-LoRA
  Serving", packed MoE LoRA loader table: 37 248 tensors become 672, declared
  bytes nearly unchanged) so that loading touches few objects.  Admitting a
  revision L_r into a GPU batch slot ("Shared-Base Rollout and Serving": the
  cold path ends with "admit L_r into a GPU batch slot") then means copying one
  stacked tensor pair per projection into the slot of a pool whose slots are
  allocated at a configured maximum rank ("Time-Sliced Multi-LoRA Training":
  smaller adapters are padded).  The copy below is that definition written out
  element by element; padding is left as it was.

* Slot residency.  The GPU-batch tier holds at most a bounded number of
  distinct adapters, promoted by the batch scheduler and released at the end of
  a step (cache-tier table of "Scale Out: Policy-Population Serving"); the
  service tracks pinned adapters ("Worker admission and eviction").  The paper
  names LRU for the CPU tier only; applying least-recently-used order to the
  slots that no running step pins is this build's reading.  LruSlots is that
  policy as a list: front = least recently used.
"""
from __future__ import annotations

from typing import List, Optional, Tuple

import numpy as np


def admit_packed_dense(A_pool: np.ndarray, B_pool: np.ndarray, slot: int, A_src: np.ndarray, B_src: np.ndarray,
                       rank: int) -> None:
    """Rank-major pool A[slot][r_max][d], B[slot][r_max][n]; source A_src[rank][d], B_src[rank][n]."""
    S, r_max, d = A_pool.shape
    n = B_pool.shape[2]
    assert 0 <= slot < S and 1 <= rank <= r_max
    assert A_src.shape == (rank, d) and B_src.shape == (rank, n)
    for j in range(rank):
        for i in range(d):
            A_pool[slot, j, i] = A_src[j, i]
        for o in range(n):
            B_pool[slot, j, o] = B_src[j, o]


def admit_packed_moe(A_pool: np.ndarray, B_pool: np.ndarray, slot: int, A_src: np.ndarray, B_src: np.ndarray,
                     rank: int) -> None:
    """Packed pool A[slot][E][d][r_max], B[slot][E][r_max][n]; source stacked along the
    expert axis: A_src[E][d][rank], B_src[E][rank][n]."""
    S, E, d, r_max = A_pool.shape
    n = B_pool.shape[3]
    assert 0 <= slot < S and 1 <= rank <= r_max
    assert A_src.shape == (E, d, rank) and B_src.shape == (E, rank, n)
    for e in range(E):
        for i in range(d):
            for j in range(rank):
                A_pool[slot, e, i, j] = A_src[e, i, j]
        for j in range(rank):
            B_pool[slot, e, j, :] = B_src[e, j, :]


class LruSlots:
    """Least-recently-used residency over num_slots slots with pins.

    acquire(id) -> (slot, admitted, evicted_id): a resident id keeps its slot
    (admitted False) and becomes most recently used; otherwise it takes the
    lowest-numbered empty slot, or the slot of the least recently used id that
    is not pinned (evicted_id names it), and admitted is True.  Every acquire
    pins the id once; release(id) removes one pin.  Raises LookupError when
    every slot is pinned."""

    def __init__(self, num_slots: int):
        self.num_slots = num_slots
        self.slot_of = {}             # id -> slot
        self.order: List[int] = []    # ids, least recently used first
        self.pins = {}                # id -> pin count

    def acquire(self, cid: int) -> Tuple[int, bool, Optional[int]]:
        if cid in self.slot_of:
            self.order.remove(cid)
            self.order.append(cid)
            self.pins[cid] = self.pins.get(cid, 0) + 1
            return self.slot_of[cid], False, None
        used = set(self.slot_of.values())
        evicted = None
        slot = None
        for s in range(self.num_slots):
            if s not in used:
                slot = s
                break
        if slot is None:
            for victim in self.order:
                if self.pins.get(victim, 0) == 0:
                    evicted = victim
                    break
            if evicted is None:
                raise LookupError("every slot is pinned")
            slot = self.slot_of.pop(evicted)
            self.order.remove(evicted)
            self.pins.pop(evicted, None)
        self.slot_of[cid] = slot
        self.order.append(cid)
        self.pins[cid] = 1
        return slot, True, evicted

    def release(self, cid: int) -> None:
        if self.pins.get(cid, 0) <= 0:
            raise KeyError(cid)
        self.pins[cid] -= 1

    def resident(self):
        return dict(self.slot_of)

"""Thin Python binding of libmint_lora.so (the C ABI in include/mint_lora.h).

Argument marshalling only: every step of the LoRA apply runs in the CUDA
library.  PyTorch supplies device memory and the stream.  There is no CPU
fallback: if the library is missing, importing it here raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# MINT_LORA_LIBRARY names another build of the same library (a debug or instrumented one).
LIB_PATH = os.environ.get("MINT_LORA_LIBRARY") or os.path.join(_PKG, "libmint_lora.so")

MINT_OK = 0
MINT_ERR_INVALID_ARG = -1
MINT_ERR_NOT_RESIDENT = -2
MINT_ERR_SHAPE_MISMATCH = -3
MINT_ERR_RANK_TOO_LARGE = -4
MINT_ERR_WORKSPACE_TOO_SMALL = -5
MINT_ERR_MISALIGNED = -6
MINT_ERR_CUDA = -7
MINT_ERR_TIMEOUT = -8
MINT_ERR_UNSUPPORTED = -9
MINT_ERR_STALE_PLAN = -10
MINT_ERR_BAD_INDEX = -11
MINT_STATUS_WORDS = 4
MINT_LAYOUT_RANK_MAJOR = 0
MINT_LAYOUT_PACKED_MOE = 1

# Every symbol include/mint_lora.h declares (the CPU test checks the export list).
EXPORTS = [
    "mint_last_error_string", "mint_status_name",
    "mint_pool_create", "mint_pool_destroy", "mint_pool_write_slot", "mint_pool_admit_packed",
    "mint_slot_manager_create", "mint_slot_manager_destroy", "mint_slot_manager_acquire",
    "mint_slot_manager_release", "mint_slot_manager_lookup",
    "mint_slot_table_create", "mint_slot_table_bind", "mint_slot_table_bind_many",
    "mint_slot_table_evict", "mint_slot_table_destroy", "mint_slot_table_generation",
    "mint_lora_plan_bytes", "mint_lora_plan_layout", "mint_lora_plan", "mint_plan_fetch_summary",
    "mint_lora_shrink", "mint_lora_expand",
    "mint_lora_apply_workspace_bytes", "mint_lora_apply_fused", "mint_lora_apply_fused_grouped",
    "mint_lora_apply_fused_static", "mint_selftest_wait_timeout",
    "mint_lora_backward_workspace_bytes", "mint_lora_backward", "mint_lora_backward_grouped",
    "mint_moe_lora_apply_workspace_bytes", "mint_moe_lora_apply", "mint_moe_lora_apply_grouped",
    "mint_moe_lora_apply_combine_workspace_bytes", "mint_moe_lora_apply_combine",
    "mint_moe_lora_backward_workspace_bytes", "mint_moe_lora_backward",
]


class MintError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{status_name(status)} ({status}): {message}")
        self.status = status


class PoolDesc(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("n", ctypes.c_int32), ("r_max", ctypes.c_int32),
                ("num_slots", ctypes.c_int32), ("num_experts", ctypes.c_int32),
                ("layout", ctypes.c_int32), ("A_dev", ctypes.c_void_p), ("B_dev", ctypes.c_void_p)]


class ApplyItem(ctypes.Structure):
    _fields_ = [("pool", ctypes.c_void_p), ("x_dev", ctypes.c_void_p), ("ldx", ctypes.c_int64),
                ("y_dev", ctypes.c_void_p), ("ldy", ctypes.c_int64), ("workspace_dev", ctypes.c_void_p),
                ("workspace_bytes", ctypes.c_size_t)]


class BackwardItem(ctypes.Structure):
    _fields_ = [("pool", ctypes.c_void_p), ("x_dev", ctypes.c_void_p), ("ldx", ctypes.c_int64),
                ("dy_dev", ctypes.c_void_p), ("lddy", ctypes.c_int64), ("dx_dev", ctypes.c_void_p),
                ("lddx", ctypes.c_int64), ("dA_dev", ctypes.c_void_p), ("dB_dev", ctypes.c_void_p),
                ("workspace_dev", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


MINT_MAX_GROUP = 8


class PlanLayout(ctypes.Structure):
    _fields_ = [("total_bytes", ctypes.c_int64), ("header_off", ctypes.c_int64),
                ("perm_off", ctypes.c_int64), ("seg_start_off", ctypes.c_int64),
                ("seg_key_off", ctypes.c_int64)]


class PlanSummary(ctypes.Structure):
    _fields_ = [("num_items", ctypes.c_int32), ("num_active", ctypes.c_int32),
                ("num_segments", ctypes.c_int32), ("max_segment", ctypes.c_int32),
                ("sum_rank", ctypes.c_int32), ("not_resident", ctypes.c_int32),
                ("bad_expert", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("generation", ctypes.c_int64)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libmint_lora.so from the package directory.  Raises when it has not
    been built (python -m paper_2605_13779_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with "
                          "`python -m paper_2605_13779_b200.build` (there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
    sig = {
        "mint_last_error_string": (ctypes.c_char_p, []),
        "mint_status_name": (ctypes.c_char_p, [i32]),
        "mint_pool_create": (i32, [ctypes.POINTER(vp), ctypes.POINTER(PoolDesc)]),
        "mint_pool_destroy": (i32, [vp]),
        "mint_pool_write_slot": (i32, [vp, i32, i32, vp, vp, i32, i32, vp]),
        "mint_pool_admit_packed": (i32, [vp, i32, vp, vp, i32, vp]),
        "mint_slot_manager_create": (i32, [ctypes.POINTER(vp), i32, vp]),
        "mint_slot_manager_destroy": (i32, [vp]),
        "mint_slot_manager_acquire": (i32, [vp, i64, i32, f32, ctypes.POINTER(i32), ctypes.POINTER(i32),
                                            ctypes.POINTER(i64), vp]),
        "mint_slot_manager_release": (i32, [vp, i64]),
        "mint_slot_manager_lookup": (i32, [vp, i64]),
        "mint_slot_table_create": (i32, [ctypes.POINTER(vp), i64, i32, vp, vp, vp, vp]),
        "mint_slot_table_bind": (i32, [vp, i64, i32, i32, f32, vp]),
        "mint_slot_table_bind_many": (i32, [vp, i64, vp, vp, vp, vp, vp]),
        "mint_slot_table_evict": (i32, [vp, i64, vp]),
        "mint_slot_table_destroy": (i32, [vp]),
        "mint_slot_table_generation": (i64, [vp]),
        "mint_lora_plan_bytes": (sz, [i32, i32, i32, i32]),
        "mint_lora_plan_layout": (i32, [i32, i32, i32, i32, ctypes.POINTER(PlanLayout)]),
        "mint_lora_plan": (i32, [vp, vp, i32, vp, i32, i32, vp, sz, vp, vp]),
        "mint_plan_fetch_summary": (i32, [vp, ctypes.POINTER(PlanSummary), vp]),
        "mint_lora_shrink": (i32, [vp, vp, vp, i32, vp, i64, vp, vp, vp]),
        "mint_lora_expand": (i32, [vp, vp, vp, i32, vp, vp, i64, vp, vp]),
        "mint_lora_apply_workspace_bytes": (sz, [vp, i32]),
        "mint_lora_apply_fused": (i32, [vp, vp, vp, i32, vp, i64, vp, i64, vp, sz, vp, vp]),
        "mint_lora_apply_fused_grouped": (i32, [ctypes.POINTER(ApplyItem), i32, vp, vp, i32, vp, vp]),
        "mint_lora_apply_fused_static": (i32, [vp, vp, vp, i32, vp, i64, vp, i64, vp, vp]),
        "mint_selftest_wait_timeout": (i32, [vp, vp, vp, i32, vp, i64, vp, sz, vp, vp]),
        "mint_moe_lora_apply_workspace_bytes": (sz, [vp, i32, i32]),
        "mint_lora_backward_workspace_bytes": (sz, [vp, i32]),
        "mint_lora_backward": (i32, [vp, vp, vp, i32, vp, i64, vp, i64, vp, i64, vp, vp, vp, sz, vp, vp]),
        "mint_lora_backward_grouped": (i32, [ctypes.POINTER(BackwardItem), i32, vp, vp, i32, vp, vp]),
        "mint_moe_lora_apply": (i32, [vp, vp, vp, i32, i32, vp, i64, i64, vp, vp, vp, i64, vp, sz, vp, vp]),
        "mint_moe_lora_apply_grouped": (i32, [ctypes.POINTER(ApplyItem), i32, vp, vp, i32, i32, i64, vp, vp, vp, vp]),
        "mint_moe_lora_apply_combine_workspace_bytes": (sz, [vp, i32, i32]),
        "mint_moe_lora_apply_combine": (i32, [vp, vp, vp, i32, i32, vp, i64, i64, vp, vp, vp, i64, vp, sz, vp, vp]),
        "mint_moe_lora_backward_workspace_bytes": (sz, [vp, i32, i32]),
        "mint_moe_lora_backward": (i32, [vp, vp, vp, i32, i32, vp, i64, i64, vp, vp, vp, i64, vp, i64, vp, vp, vp, sz,
                                         vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def status_name(status: int) -> str:
    return load_library().mint_status_name(int(status)).decode()


def last_error() -> str:
    return load_library().mint_last_error_string().decode()


def _check(status: int):
    if status != MINT_OK:
        raise MintError(status, last_error())


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda, "device tensor expected"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def bf16_from_bits(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns (numpy) -> torch.bfloat16 tensor on the device."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.view(torch.bfloat16).to(device)


def bits_from_bf16(t: torch.Tensor) -> np.ndarray:
    """torch.bfloat16 tensor -> uint16 bit patterns on the host."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def new_status(device="cuda") -> torch.Tensor:
    return torch.zeros(MINT_STATUS_WORDS, dtype=torch.int32, device=device)


# --------------------------------------------------------------------------
# handles
# --------------------------------------------------------------------------
class Pool:
    """Packed weights of one projection over all GPU slots (caller-owned
    tensors A, B in bf16)."""

    def __init__(self, A: torch.Tensor, B: torch.Tensor, d: int, n: int, r_max: int, num_slots: int,
                 num_experts: int = 0, layout: Optional[int] = None):
        lib = load_library()
        if layout is None:
            layout = MINT_LAYOUT_PACKED_MOE if num_experts > 0 else MINT_LAYOUT_RANK_MAJOR
        self.A, self.B = A, B
        self.d, self.n, self.r_max, self.num_slots, self.num_experts = d, n, r_max, num_slots, num_experts
        self.layout = layout
        desc = PoolDesc(d, n, r_max, num_slots, num_experts, layout, _ptr(A), _ptr(B))
        h = ctypes.c_void_p()
        _check(lib.mint_pool_create(ctypes.byref(h), ctypes.byref(desc)))
        self.handle = h

    def write_slot(self, slot: int, A_src, B_src, rank: int, expert: int = -1):
        """A_src/B_src: torch tensors (device or pinned/pageable host), bf16."""
        lib = load_library()
        on_dev = A_src.is_cuda
        assert B_src.is_cuda == on_dev
        _check(lib.mint_pool_write_slot(self.handle, slot, expert, A_src.data_ptr(), B_src.data_ptr(),
                                        rank, 1 if on_dev else 0, _stream()))

    def admit_packed(self, slot: int, A_packed: torch.Tensor, B_packed: torch.Tensor, rank: int):
        """The stacked tensors of one adapter projection (device, bf16, contiguous) into a slot:
        [E][d][rank], [E][rank][n] for packed MoE pools; [rank][d], [rank][n] for dense pools."""
        assert A_packed.is_cuda and B_packed.is_cuda and A_packed.is_contiguous() and B_packed.is_contiguous()
        _check(load_library().mint_pool_admit_packed(self.handle, slot, _ptr(A_packed), _ptr(B_packed), rank,
                                                     _stream()))

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.mint_pool_destroy(self.handle)
            self.handle = None


class SlotTable:
    """Catalog id -> slot and per-slot (rank, scale); device arrays are torch
    tensors owned here, the host mirror lives in the library handle."""

    def __init__(self, catalog_size: int, num_slots: int, device="cuda"):
        lib = load_library()
        self.catalog_size, self.num_slots = catalog_size, num_slots
        self.id_to_slot = torch.empty(catalog_size, dtype=torch.int32, device=device)
        self.slot_rank = torch.empty(num_slots, dtype=torch.int32, device=device)
        self.slot_scale = torch.empty(num_slots, dtype=torch.float32, device=device)
        h = ctypes.c_void_p()
        _check(lib.mint_slot_table_create(ctypes.byref(h), catalog_size, num_slots, _ptr(self.id_to_slot),
                                          _ptr(self.slot_rank), _ptr(self.slot_scale), _stream()))
        self.handle = h

    def bind(self, catalog_id: int, slot: int, rank: int, scale: float):
        _check(load_library().mint_slot_table_bind(self.handle, catalog_id, slot, rank, scale, _stream()))

    def bind_many(self, ids, slots, ranks, scales):
        ids = np.ascontiguousarray(ids, dtype=np.int64)
        slots = np.ascontiguousarray(slots, dtype=np.int32)
        ranks = np.ascontiguousarray(ranks, dtype=np.int32)
        scales = np.ascontiguousarray(scales, dtype=np.float32)
        assert ids.shape == slots.shape == ranks.shape == scales.shape
        _check(load_library().mint_slot_table_bind_many(
            self.handle, ids.shape[0], ids.ctypes.data, slots.ctypes.data, ranks.ctypes.data,
            scales.ctypes.data, _stream()))

    def evict(self, catalog_id: int):
        _check(load_library().mint_slot_table_evict(self.handle, catalog_id, _stream()))

    @property
    def generation(self) -> int:
        return int(load_library().mint_slot_table_generation(self.handle))

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.mint_slot_table_destroy(self.handle)
            self.handle = None


class SlotManager:
    """Which adapters hold the GPU slots: least-recently-used order over the slots no running
    step pins.  With a table, acquire also evicts and binds in the table."""

    def __init__(self, num_slots: int, table: Optional[SlotTable] = None):
        self.table = table
        h = ctypes.c_void_p()
        _check(load_library().mint_slot_manager_create(ctypes.byref(h), num_slots,
                                                       table.handle if table is not None else None))
        self.handle = h

    def acquire(self, catalog_id: int, rank: int = 1, scale: float = 1.0):
        """-> (slot, admitted, evicted id or None); pins the id once."""
        slot, admitted, evicted = ctypes.c_int32(-1), ctypes.c_int32(0), ctypes.c_int64(-1)
        stream = _stream() if self.table is not None else None
        _check(load_library().mint_slot_manager_acquire(self.handle, catalog_id, rank, scale, ctypes.byref(slot),
                                                        ctypes.byref(admitted), ctypes.byref(evicted), stream))
        return slot.value, bool(admitted.value), (None if evicted.value < 0 else evicted.value)

    def release(self, catalog_id: int):
        _check(load_library().mint_slot_manager_release(self.handle, catalog_id))

    def lookup(self, catalog_id: int) -> int:
        return int(load_library().mint_slot_manager_lookup(self.handle, catalog_id))

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.mint_slot_manager_destroy(self.handle)
            self.handle = None


class Plan:
    """The opaque device plan blob plus the shape it was made for."""

    def __init__(self, T: int, K: int, num_slots: int, num_experts: int, device="cuda"):
        lib = load_library()
        self.T, self.K, self.num_slots, self.num_experts = T, K, num_slots, num_experts
        self.layout = PlanLayout()
        _check(lib.mint_lora_plan_layout(T, K, num_slots, num_experts, ctypes.byref(self.layout)))
        self.nbytes = int(lib.mint_lora_plan_bytes(T, K, num_slots, num_experts))
        assert self.nbytes == self.layout.total_bytes
        self.blob = torch.empty(self.nbytes, dtype=torch.uint8, device=device)

    def summary(self) -> PlanSummary:
        s = PlanSummary()
        _check(load_library().mint_plan_fetch_summary(_ptr(self.blob), ctypes.byref(s), _stream()))
        return s

    def arrays(self) -> dict:
        """Canonical plan arrays on the host (synchronises): perm, seg_start, seg_key."""
        s = self.summary()
        host = self.blob.cpu().numpy()

        def take(off, count):
            return host[off:off + 4 * count].view(np.int32).copy()
        return {
            "perm": take(self.layout.perm_off, s.num_active),
            "seg_start": take(self.layout.seg_start_off, s.num_segments + 1),
            "seg_key": take(self.layout.seg_key_off, s.num_segments),
            "S": s.num_segments,
            "n_active": s.num_active,
            "n_not_resident": s.not_resident,
            "n_bad_expert": s.bad_expert,
            "max_segment": s.max_segment,
            "sum_rank": s.sum_rank,
        }


# --------------------------------------------------------------------------
# calls (same names as the C ABI)
# --------------------------------------------------------------------------
def mint_lora_plan(table: SlotTable, ids: torch.Tensor, status: torch.Tensor,
                   expert_ids: Optional[torch.Tensor] = None, num_experts: int = 0,
                   plan: Optional[Plan] = None) -> Plan:
    assert ids.dtype == torch.int64 and ids.is_contiguous()
    T = ids.shape[0]
    K = 1
    if expert_ids is not None:
        assert expert_ids.dtype == torch.int32 and expert_ids.is_contiguous()
        K = expert_ids.shape[1] if expert_ids.dim() == 2 else 1
    if plan is None:
        plan = Plan(T, K, table.num_slots, num_experts, device=ids.device)
    _check(load_library().mint_lora_plan(table.handle, _ptr(ids) if T else None, T, _ptr(expert_ids), K,
                                         num_experts, _ptr(plan.blob), plan.nbytes, _ptr(status), _stream()))
    return plan


def mint_lora_shrink(pool: Pool, table: SlotTable, plan: Plan, x: torch.Tensor, status: torch.Tensor,
                     v: Optional[torch.Tensor] = None) -> torch.Tensor:
    if v is None:
        v = torch.empty(plan.T, pool.r_max, dtype=torch.float32, device=x.device)
    assert v.dtype == torch.float32 and v.is_contiguous()
    _check(load_library().mint_lora_shrink(pool.handle, table.handle, _ptr(plan.blob), plan.T, _ptr(x),
                                           x.stride(0) if x.dim() == 2 and x.shape[0] > 0 else pool.d,
                                           _ptr(v), _ptr(status), _stream()))
    return v


def mint_lora_expand(pool: Pool, table: SlotTable, plan: Plan, v: torch.Tensor, y: torch.Tensor,
                     status: torch.Tensor) -> torch.Tensor:
    _check(load_library().mint_lora_expand(pool.handle, table.handle, _ptr(plan.blob), plan.T, _ptr(v),
                                           _ptr(y), y.stride(0) if y.dim() == 2 and y.shape[0] > 0 else pool.n,
                                           _ptr(status), _stream()))
    return y


def mint_lora_apply_workspace_bytes(pool: Pool, T: int) -> int:
    return int(load_library().mint_lora_apply_workspace_bytes(pool.handle, T))


def new_workspace(pool: Pool, T: int, device="cuda") -> torch.Tensor:
    """Workspace of the fused apply for one projection; it needs no initialisation
    (every call writes each entry before it reads it)."""
    nbytes = max(256, mint_lora_apply_workspace_bytes(pool, T))
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def _ld(t: torch.Tensor, width: int) -> int:
    return t.stride(0) if t.dim() == 2 and t.shape[0] > 0 else width


def mint_lora_apply_fused(pool: Pool, table: SlotTable, plan: Plan, x: torch.Tensor, y: torch.Tensor,
                          status: torch.Tensor, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    if workspace is None:
        workspace = new_workspace(pool, plan.T, x.device)
    _check(load_library().mint_lora_apply_fused(
        pool.handle, table.handle, _ptr(plan.blob), plan.T, _ptr(x), _ld(x, pool.d), _ptr(y), _ld(y, pool.n),
        _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status), _stream()))
    return y


MINT_STATIC_WORKSPACE_BYTES = 8 << 20


def mint_lora_apply_fused_static(pool: Pool, table: SlotTable, plan: Plan, x: torch.Tensor, y: torch.Tensor,
                                 status: torch.Tensor) -> torch.Tensor:
    """The fused apply with the library's built-in workspace: no workspace tensor
    is passed and nothing is allocated.  For callers that cannot allocate device
    memory; batches that need more than MINT_STATIC_WORKSPACE_BYTES are refused.
    Calls share the built-in workspace, so keep them ordered on one stream."""
    _check(load_library().mint_lora_apply_fused_static(
        pool.handle, table.handle, _ptr(plan.blob), plan.T, _ptr(x), _ld(x, pool.d), _ptr(y), _ld(y, pool.n),
        _ptr(status), _stream()))
    return y


def mint_selftest_wait_timeout(pool: Pool, table: SlotTable, plan: Plan, x: torch.Tensor, status: torch.Tensor,
                               workspace: torch.Tensor):
    """Runs the dense-segment shrink with its tensor-core work withheld: its bounded waits run out."""
    _check(load_library().mint_selftest_wait_timeout(
        pool.handle, table.handle, _ptr(plan.blob), plan.T, _ptr(x), _ld(x, pool.d), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(status), _stream()))


class ApplyGroup:
    """Up to MINT_MAX_GROUP (pool, x, y, workspace) items sharing one plan, marshalled once."""

    def __init__(self, items):
        assert 1 <= len(items) <= MINT_MAX_GROUP
        self.keep = items
        arr = (ApplyItem * len(items))()
        for i, (pool, x, y, ws) in enumerate(items):
            arr[i] = ApplyItem(pool.handle, _ptr(x), _ld(x, pool.d), _ptr(y), _ld(y, pool.n), _ptr(ws),
                               ws.numel() * ws.element_size())
        self.array = arr
        self.count = len(items)


def mint_lora_apply_fused_grouped(group: ApplyGroup, table: SlotTable, plan: Plan, status: torch.Tensor):
    _check(load_library().mint_lora_apply_fused_grouped(group.array, group.count, table.handle,
                                                        _ptr(plan.blob), plan.T, _ptr(status), _stream()))


def new_backward_workspace(pool: Pool, T: int, device="cuda") -> torch.Tensor:
    """Workspace of the backward for one projection; it needs no initialisation."""
    nbytes = max(256, int(load_library().mint_lora_backward_workspace_bytes(pool.handle, T)))
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def mint_lora_backward(pool: Pool, table: SlotTable, plan: Plan, x: torch.Tensor, dy: torch.Tensor,
                       status: torch.Tensor, dx: Optional[torch.Tensor] = None,
                       dA: Optional[torch.Tensor] = None, dB: Optional[torch.Tensor] = None,
                       workspace: Optional[torch.Tensor] = None):
    """dx (bf16 [T, d]) and dA / dB (fp32, shaped like the pool's tensors) are accumulated into."""
    for g in (dA, dB):
        assert g is None or (g.dtype == torch.float32 and g.is_contiguous())
    if workspace is None:
        workspace = new_backward_workspace(pool, plan.T, device=x.device)
    _check(load_library().mint_lora_backward(
        pool.handle, table.handle, _ptr(plan.blob), plan.T, _ptr(x), _ld(x, pool.d), _ptr(dy), _ld(dy, pool.n),
        _ptr(dx), _ld(dx, pool.d) if dx is not None else 0, _ptr(dA), _ptr(dB), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(status), _stream()))


class BackwardGroup:
    """Up to MINT_MAX_GROUP (pool, x, dy, dx, dA, dB, workspace) items sharing one plan, marshalled once;
    dx, or dA and dB together, may be None."""

    def __init__(self, items):
        assert 1 <= len(items) <= MINT_MAX_GROUP
        self.keep = items
        arr = (BackwardItem * len(items))()
        for i, (pool, x, dy, dx, dA, dB, ws) in enumerate(items):
            for g in (dA, dB):
                assert g is None or (g.dtype == torch.float32 and g.is_contiguous())
            arr[i] = BackwardItem(pool.handle, _ptr(x), _ld(x, pool.d), _ptr(dy), _ld(dy, pool.n), _ptr(dx),
                                  _ld(dx, pool.d) if dx is not None else 0, _ptr(dA), _ptr(dB), _ptr(ws),
                                  ws.numel() * ws.element_size())
        self.array = arr
        self.count = len(items)


def mint_lora_backward_grouped(group: BackwardGroup, table: SlotTable, plan: Plan, status: torch.Tensor):
    _check(load_library().mint_lora_backward_grouped(group.array, group.count, table.handle, _ptr(plan.blob),
                                                     plan.T, _ptr(status), _stream()))


def mint_moe_lora_apply_workspace_bytes(pool: Pool, T: int, K: int) -> int:
    return int(load_library().mint_moe_lora_apply_workspace_bytes(pool.handle, T, K))


def new_moe_workspace(pool: Pool, T: int, K: int, device="cuda") -> torch.Tensor:
    """Workspace of the MoE apply for one projection; it needs no initialisation."""
    nbytes = max(256, mint_moe_lora_apply_workspace_bytes(pool, T, K))
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def mint_moe_lora_apply(pool: Pool, table: SlotTable, plan: Plan, x: torch.Tensor, y: torch.Tensor,
                        status: torch.Tensor, x_row: Optional[torch.Tensor] = None,
                        pair_weight: Optional[torch.Tensor] = None,
                        workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    if x_row is not None:
        assert x_row.dtype == torch.int32 and x_row.is_contiguous()
    if pair_weight is not None:
        assert pair_weight.dtype == torch.float32 and pair_weight.is_contiguous()
    if workspace is None:
        workspace = new_moe_workspace(pool, plan.T, plan.K, device=y.device)
    _check(load_library().mint_moe_lora_apply(
        pool.handle, table.handle, _ptr(plan.blob), plan.T, plan.K, _ptr(x), x.stride(0), x.shape[0],
        _ptr(x_row), _ptr(pair_weight), _ptr(y), y.stride(0),
        _ptr(workspace), workspace.numel() * workspace.element_size() if workspace is not None else 0,
        _ptr(status), _stream()))
    return y


def mint_moe_lora_apply_grouped(items, table: SlotTable, plan: Plan, status: torch.Tensor,
                                x_row: Optional[torch.Tensor] = None,
                                pair_weight: Optional[torch.Tensor] = None):
    """items: (pool, x, y, workspace) per projection (the item record has the layout of the dense one);
    they share the plan, the row map and the pair weights."""
    assert 1 <= len(items) <= MINT_MAX_GROUP
    if x_row is not None:
        assert x_row.dtype == torch.int32 and x_row.is_contiguous()
    if pair_weight is not None:
        assert pair_weight.dtype == torch.float32 and pair_weight.is_contiguous()
    arr = (ApplyItem * len(items))()
    for i, (pool, x, y, ws) in enumerate(items):
        arr[i] = ApplyItem(pool.handle, _ptr(x), x.stride(0), _ptr(y), y.stride(0), _ptr(ws),
                           ws.numel() * ws.element_size())
    _check(load_library().mint_moe_lora_apply_grouped(
        arr, len(items), table.handle, _ptr(plan.blob), plan.T, plan.K, items[0][1].shape[0],
        _ptr(x_row), _ptr(pair_weight), _ptr(status), _stream()))


def mint_moe_lora_apply_combine(pool: Pool, table: SlotTable, plan: Plan, x: torch.Tensor, y: torch.Tensor,
                                status: torch.Tensor, pair_weight: torch.Tensor,
                                x_row: Optional[torch.Tensor] = None,
                                workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """y: [T][n], updated in place with the router-weighted sum over each token's K experts."""
    assert pair_weight.dtype == torch.float32 and pair_weight.is_contiguous()
    if x_row is not None:
        assert x_row.dtype == torch.int32 and x_row.is_contiguous()
    lib = load_library()
    if workspace is None:
        nbytes = max(256, int(lib.mint_moe_lora_apply_combine_workspace_bytes(pool.handle, plan.T, plan.K)))
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=y.device)
    _check(lib.mint_moe_lora_apply_combine(
        pool.handle, table.handle, _ptr(plan.blob), plan.T, plan.K, _ptr(x), x.stride(0), x.shape[0],
        _ptr(x_row), _ptr(pair_weight), _ptr(y), y.stride(0), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(status), _stream()))
    return y


def mint_moe_lora_backward(pool: Pool, table: SlotTable, plan: Plan, x: torch.Tensor, dy: torch.Tensor,
                           status: torch.Tensor, dx: Optional[torch.Tensor] = None,
                           dA: Optional[torch.Tensor] = None, dB: Optional[torch.Tensor] = None,
                           x_row: Optional[torch.Tensor] = None, pair_weight: Optional[torch.Tensor] = None,
                           workspace: Optional[torch.Tensor] = None):
    """dx (bf16 [T*K, d], one row per pair) and dA / dB (fp32, shaped like the pool's packed tensors)
    are accumulated into; dy is bf16 [T*K, n]."""
    if x_row is not None:
        assert x_row.dtype == torch.int32 and x_row.is_contiguous()
    if pair_weight is not None:
        assert pair_weight.dtype == torch.float32 and pair_weight.is_contiguous()
    for g in (dA, dB):
        assert g is None or (g.dtype == torch.float32 and g.is_contiguous())
    lib = load_library()
    if workspace is None:
        nbytes = max(256, int(lib.mint_moe_lora_backward_workspace_bytes(pool.handle, plan.T, plan.K)))
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=dy.device)
    _check(lib.mint_moe_lora_backward(
        pool.handle, table.handle, _ptr(plan.blob), plan.T, plan.K, _ptr(x), x.stride(0), x.shape[0],
        _ptr(x_row), _ptr(pair_weight), _ptr(dy), dy.stride(0), _ptr(dx), dx.stride(0) if dx is not None else 0,
        _ptr(dA), _ptr(dB), _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status), _stream()))
    return dx, dA, dB

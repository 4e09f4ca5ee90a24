"""The C-ABI library loads without a GPU, exports every declared symbol, and
its host-side validation rejects bad arguments before any launch (CPU only)."""
import ctypes
import os
import re

import pytest

from paper_2605_13779_b200 import build as mint_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    mint_build.build()
    from paper_2605_13779_b200 import binding
    return binding, binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    binding, l = lib
    header = open(os.path.join(ROOT, "include", "mint_lora.h")).read()
    declared = set(re.findall(r"\b(mint_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(l, name) is not None


def test_status_names(lib):
    binding, _ = lib
    assert binding.status_name(0) == "MINT_OK"
    assert binding.status_name(-2) == "MINT_ERR_NOT_RESIDENT"
    assert binding.status_name(-10) == "MINT_ERR_STALE_PLAN"


def test_plan_bytes_and_layout(lib):
    binding, l = lib
    lay = binding.PlanLayout()
    assert l.mint_lora_plan_layout(256, 1, 64, 0, ctypes.byref(lay)) == 0
    assert lay.total_bytes == l.mint_lora_plan_bytes(256, 1, 64, 0) > 0
    assert 0 <= lay.header_off < lay.perm_off < lay.seg_start_off < lay.seg_key_off < lay.total_bytes
    assert lay.perm_off % 16 == 0 and lay.seg_start_off % 16 == 0
    assert l.mint_lora_plan_bytes(0, 1, 4, 0) > 0                # an empty batch still has a header
    assert l.mint_lora_plan_bytes(-1, 1, 4, 0) == 0
    assert l.mint_lora_plan_layout(4, 0, 4, 0, ctypes.byref(lay)) == binding.MINT_ERR_INVALID_ARG
    assert l.mint_lora_plan_layout(1 << 20, 64, 4, 0, ctypes.byref(lay)) == binding.MINT_ERR_UNSUPPORTED


@pytest.mark.parametrize("kw,code", [
    (dict(d=2561), "MINT_ERR_SHAPE_MISMATCH"),
    (dict(n=100), "MINT_ERR_SHAPE_MISMATCH"),
    (dict(r_max=0), "MINT_ERR_INVALID_ARG"),
    (dict(r_max=4096), "MINT_ERR_RANK_TOO_LARGE"),
    (dict(A=0), "MINT_ERR_INVALID_ARG"),
    (dict(A=4104), "MINT_ERR_MISALIGNED"),
    (dict(layout=7), "MINT_ERR_INVALID_ARG"),
    (dict(layout=0, num_experts=4), "MINT_ERR_UNSUPPORTED"),
    (dict(layout=1, num_experts=0), "MINT_ERR_INVALID_ARG"),
])
def test_pool_create_validation(lib, kw, code):
    binding, l = lib
    args = dict(d=64, n=64, r_max=8, num_slots=4, num_experts=0, layout=0, A=4096, B=8192)
    args.update(kw)
    desc = binding.PoolDesc(args["d"], args["n"], args["r_max"], args["num_slots"], args["num_experts"],
                            args["layout"], args["A"], args["B"])
    h = ctypes.c_void_p()
    st = l.mint_pool_create(ctypes.byref(h), ctypes.byref(desc))
    assert binding.status_name(st) == code
    assert h.value is None
    assert binding.last_error() != ""


def test_pool_create_and_destroy_without_device(lib):
    binding, l = lib
    desc = binding.PoolDesc(64, 128, 8, 4, 0, 0, 4096, 8192)
    h = ctypes.c_void_p()
    assert l.mint_pool_create(ctypes.byref(h), ctypes.byref(desc)) == 0
    assert h.value
    assert l.mint_pool_destroy(h) == 0


def test_null_arguments_are_rejected(lib):
    binding, l = lib
    assert l.mint_lora_plan(None, None, 4, None, 1, 0, None, 0, None, None) == binding.MINT_ERR_INVALID_ARG
    assert l.mint_lora_apply_fused(None, None, None, 4, None, 8, None, 8, None, 0, None, None) == binding.MINT_ERR_INVALID_ARG
    assert l.mint_moe_lora_apply(None, None, None, 4, 2, None, 8, 8, None, None, None, 8, None, 0, None, None) == binding.MINT_ERR_INVALID_ARG
    assert l.mint_slot_table_evict(None, 0, None) == binding.MINT_ERR_INVALID_ARG


def test_slot_manager_without_a_table_follows_the_oracle_model(lib):
    """The library's slot manager (bookkeeping only, no GPU) against the plain model and the
    hand-worked sequence."""
    import random
    from oracle import admission
    import test_oracle_admission as golden
    binding, _ = lib
    m = binding.SlotManager(3)
    for op in golden.read_lru_golden():
        if op[0] == "acquire":
            assert m.acquire(op[1]) == (op[2], op[3], op[4]), op
        elif op[0] == "release":
            m.release(op[1])
        else:
            with pytest.raises(binding.MintError) as e:
                m.acquire(op[1])
            assert e.value.status == binding.MINT_ERR_NOT_RESIDENT
    rnd = random.Random(5)
    m, o, held = binding.SlotManager(7), admission.LruSlots(7), []
    for step in range(5000):
        if held and rnd.random() < 0.45:
            c = held.pop(rnd.randrange(len(held)))
            m.release(c)
            o.release(c)
            continue
        c = rnd.randrange(1_000_000) if rnd.random() < 0.3 else rnd.randrange(20)
        try:
            want = o.acquire(c)
        except LookupError:
            want = None
        try:
            got = m.acquire(c)
        except binding.MintError:
            got = None
        assert got == want, (step, c, got, want)
        if got:
            held.append(c)
        assert m.lookup(c) == (got[0] if got else o.resident().get(c, -1))
    with pytest.raises(binding.MintError):
        m.release(123456789)

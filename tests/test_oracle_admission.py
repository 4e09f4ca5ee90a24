"""Pins of the admission oracle (oracle/admission.py): the packed copy against
numpy slicing and a hand example, the slot residency model against a sequence
worked by hand and against its invariants."""
import os

import numpy as np
import pytest

from oracle import admission

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def test_packed_moe_copy_equals_slicing_and_leaves_padding():
    rng = np.random.default_rng(3)
    S, E, d, n, r_max, rank = 3, 4, 5, 6, 4, 3
    A = rng.integers(0, 60000, size=(S, E, d, r_max)).astype(np.uint16)
    B = rng.integers(0, 60000, size=(S, E, r_max, n)).astype(np.uint16)
    A0, B0 = A.copy(), B.copy()
    As = rng.integers(0, 60000, size=(E, d, rank)).astype(np.uint16)
    Bs = rng.integers(0, 60000, size=(E, rank, n)).astype(np.uint16)
    admission.admit_packed_moe(A, B, 1, As, Bs, rank)
    np.testing.assert_array_equal(A[1, :, :, :rank], As)
    np.testing.assert_array_equal(B[1, :, :rank, :], Bs)
    np.testing.assert_array_equal(A[1, :, :, rank:], A0[1, :, :, rank:])     # padding untouched
    np.testing.assert_array_equal(B[1, :, rank:, :], B0[1, :, rank:, :])
    for s in (0, 2):                                                          # other slots untouched
        np.testing.assert_array_equal(A[s], A0[s])
        np.testing.assert_array_equal(B[s], B0[s])


def test_packed_moe_copy_hand_example():
    """E=2, d=2, r_max=2, rank=1, n=1: element (e, i, 0) of the source lands at flat index
    ((slot*E + e)*d + i)*r_max of A, element (e, 0, 0) at (slot*E + e)*r_max*n of B."""
    A = np.zeros((2, 2, 2, 2), dtype=np.uint16)
    B = np.zeros((2, 2, 2, 1), dtype=np.uint16)
    As = np.array([[[1], [2]], [[3], [4]]], dtype=np.uint16)
    Bs = np.array([[[7]], [[9]]], dtype=np.uint16)
    admission.admit_packed_moe(A, B, 1, As, Bs, 1)
    assert A.reshape(-1).tolist() == [0] * 8 + [1, 0, 2, 0, 3, 0, 4, 0]
    assert B.reshape(-1).tolist() == [0] * 4 + [7, 0, 9, 0]


def test_dense_copy_equals_slicing():
    rng = np.random.default_rng(4)
    A = rng.integers(0, 60000, size=(2, 4, 7)).astype(np.uint16)
    B = rng.integers(0, 60000, size=(2, 4, 3)).astype(np.uint16)
    A0, B0 = A.copy(), B.copy()
    As = rng.integers(0, 60000, size=(2, 7)).astype(np.uint16)
    Bs = rng.integers(0, 60000, size=(2, 3)).astype(np.uint16)
    admission.admit_packed_dense(A, B, 0, As, Bs, 2)
    np.testing.assert_array_equal(A[0, :2], As)
    np.testing.assert_array_equal(B[0, :2], Bs)
    np.testing.assert_array_equal(A[0, 2:], A0[0, 2:])
    np.testing.assert_array_equal(A[1], A0[1])
    np.testing.assert_array_equal(B[1], B0[1])


def read_lru_golden():
    ops = []
    for line in open(os.path.join(GOLDEN, "lru_tiny.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w = line.split()
        if w[0] == "acquire":
            ops.append(("acquire", int(w[1]), int(w[3]), bool(int(w[4])), None if w[5] == "-" else int(w[5])))
        else:
            ops.append((w[0], int(w[1])))
    return ops


def test_lru_model_follows_the_hand_worked_sequence():
    m = admission.LruSlots(3)
    for op in read_lru_golden():
        if op[0] == "acquire":
            assert m.acquire(op[1]) == (op[2], op[3], op[4]), op
        elif op[0] == "release":
            m.release(op[1])
        else:
            with pytest.raises(LookupError):
                m.acquire(op[1])


def test_lru_model_invariants_on_random_traffic():
    """The victim is always the unpinned id whose last acquire is the oldest (checked against
    timestamps kept here), no two ids share a slot, pinned ids never lose their slot."""
    rng = np.random.default_rng(11)
    m = admission.LruSlots(5)
    last_use, pinned, clock = {}, {}, 0
    for _ in range(3000):
        clock += 1
        if pinned and rng.random() < 0.5:
            cid = list(pinned)[rng.integers(len(pinned))]
            m.release(cid)
            pinned[cid] -= 1
            if pinned[cid] == 0:
                del pinned[cid]
            continue
        cid = int(rng.integers(0, 14))
        before = m.resident()
        try:
            slot, admitted, evicted = m.acquire(cid)
        except LookupError:
            assert cid not in before and len(before) == 5 and all(c in pinned for c in before)
            continue
        assert admitted == (cid not in before)
        if evicted is not None:
            assert evicted not in pinned
            candidates = [c for c in before if c not in pinned]
            assert evicted == min(candidates, key=lambda c: last_use[c])
            assert before[evicted] == slot
        elif admitted:
            assert slot == min(set(range(5)) - set(before.values()))
        last_use[cid] = clock
        pinned[cid] = pinned.get(cid, 0) + 1
        res = m.resident()
        assert len(set(res.values())) == len(res) <= 5
        assert all(c in res for c in pinned)

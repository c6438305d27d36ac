"""The C-ABI library loads without a GPU and exports what include/sagekv.h declares."""

import ctypes
import os
import re

import pytest

from oracle import sagekv_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "sagekv.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2503_08879_b200 import build
    return ctypes.CDLL(build.build())


def declared_symbols():
    text = re.sub(r"/\*.*?\*/", "", open(HEADER).read(), flags=re.S)
    return sorted(set(re.findall(r"\b(sagekv_[a-z_]+)\s*\(", text)))


def test_header_declares_the_three_hot_calls():
    names = declared_symbols()
    for n in ("sagekv_score", "sagekv_select_compact", "sagekv_decode_attn", "sagekv_create", "sagekv_destroy"):
        assert n in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_symbols():
        assert getattr(lib, name) is not None, name


def test_strerror(lib):
    lib.sagekv_strerror.restype = ctypes.c_char_p
    assert lib.sagekv_strerror(0) == b"ok"
    texts = {lib.sagekv_strerror(c) for c in range(-9, 1)}
    assert len(texts) == 10 and lib.sagekv_strerror(-99) not in texts
    assert b"another device" in lib.sagekv_strerror(-9)          # SAGEKV_ERR_DEVICE: context used off its device


def test_status_word_maps_to_a_return_code(lib):
    """Host logic of sagekv_status: which return code a device status word gives (needs no device)."""
    code = lib.sagekv_status_code
    code.argtypes, code.restype = [ctypes.c_int32], ctypes.c_int
    assert code(0) == 0
    assert code(1) == -7                 # a bounded wait ran out: SAGEKV_ERR_TIMEOUT
    assert code(2) == -8                 # checked build found an index out of range: SAGEKV_ERR_BOUNDS
    assert code(3) == -7                 # the timeout is reported first
    assert lib.sagekv_status(None, None) == -1
    assert lib.sagekv_checked_build() == 0


def test_checked_build_compiles_and_says_so():
    from paper_2503_08879_b200 import build
    checked = ctypes.CDLL(build.build(checks=True))
    assert checked.sagekv_checked_build() == 1
    for name in declared_symbols():
        assert getattr(checked, name) is not None, name


def test_hint_and_stride_helpers_reject_bad_arguments(lib):
    lib.sagekv_scores_row_stride.restype = ctypes.c_int64
    assert lib.sagekv_set_select_hint(None, 1, 0) == -1
    assert lib.sagekv_scores_row_stride(None, ctypes.c_int64(100), 4, 16) == -1


def test_budget_split_host_function_matches_paper_and_oracle(lib):
    i32 = ctypes.c_int32
    a, b, c = i32(), i32(), i32()
    rows = [l.split() for l in open(os.path.join(ROOT, "tests", "golden", "budget_split.txt"))
            if l.strip() and l[0] != "#"]
    for B, G, sink, k, recent in (map(int, r) for r in rows):
        assert lib.sagekv_budget_split(B, G, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)) == 0
        assert (a.value, b.value, c.value) == (sink, k, recent)
    for B in (4, 64, 500, 1024, 2048, 4096, 8192, 10000):
        for G in (1, 2, 3, 4, 7, 8):
            assert lib.sagekv_budget_split(B, G, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)) == 0
            assert (a.value, b.value, c.value) == O.budget_split(B, G)
    assert lib.sagekv_budget_split(3, 4, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)) == -1
    assert lib.sagekv_budget_split(64, 0, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)) == -1
    assert lib.sagekv_budget_split(64, 4, None, ctypes.byref(b), ctypes.byref(c)) == -1


def test_null_context_is_rejected_before_any_cuda_call(lib):
    assert lib.sagekv_destroy(None) == -1
    for setter in (lib.sagekv_set_overlap, lib.sagekv_set_select_overlap, lib.sagekv_set_decode_variant, lib.sagekv_set_group_mode):
        assert setter(None, 0) == -1
    assert lib.sagekv_create(None, None, ctypes.c_int64(1), 1) == -1

"""Host-side checks of the C-ABI library that need no GPU."""
import ctypes
import os
import re

import pytest

from paper_2605_03110_b200 import build as ada_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    return ctypes.CDLL(ada_build.build())


def declared_functions():
    src = open(os.path.join(ROOT, "include", "ada.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(ada_[a-z_0-9]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"ada_create", "ada_normalize", "ada_select_full", "ada_cascade_step",
            "ada_gram_op_count", "ada_device_status"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_symbols():
    from paper_2605_03110_b200 import binding
    assert sorted(binding.SYMBOLS) == declared_functions()


def test_op_count_on_host(lib, golden):
    f = lib.ada_gram_op_count
    f.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64]
    f.restype = ctypes.c_uint64
    assert f(0, 512, 4096, 0) == 512 * 512 * 4096
    assert f(1, 512, 4096, 240) == 512 * 240 * 4096
    assert f(1, 8192, 4096, 8192) == f(0, 8192, 4096, 0)       # r = T costs the full Gram
    assert f(1, 16, 8, 17) == 0 and f(0, -1, 8, 0) == 0
    assert f(0, 16384, 4096, 0) == 16384 ** 2 * 4096           # no 32-bit overflow
    for kind, *row in golden("table7_and_cost_model.txt"):     # Table 7: L * T^2 with d = 1
        if kind == "indep":
            _, L, T, printed = row
            assert abs(int(L) * f(0, int(T), 1, 0) / 1e6 - float(printed)) < 0.006


def test_status_strings(lib):
    f = lib.ada_status_string
    f.restype = ctypes.c_char_p
    f.argtypes = [ctypes.c_int]
    assert f(0) == b"ADA_OK" and f(7) == b"ADA_ERR_TIMEOUT" and f(8) == b"ADA_ERR_BAD_TAU"
    assert len({f(i) for i in range(8)}) == 8


def test_create_rejects_bad_arguments_before_touching_a_device(lib):
    h = ctypes.c_void_p()
    f = lib.ada_create
    f.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int] + [ctypes.c_int64] * 3 + [ctypes.c_int]
    assert f(ctypes.byref(h), 0, 0, 128, 64, 0) == 1            # ADA_ERR_INVALID_ARG
    assert f(ctypes.byref(h), 0, 1, 128, 64, 5) == 1
    assert f(None, 0, 1, 128, 64, 0) == 1
    # the per-sequence list counts live in 21-bit fields: longer sequences are refused
    assert f(ctypes.byref(h), 0, 1, (1 << 21), 64, 1) == 1
    assert f(ctypes.byref(h), 0, 1 << 12, 1 << 20, 64, 1) == 1   # maxB * maxT above 2^30
    assert h.value is None

"""The C-ABI library loads on a machine without a GPU and exports every symbol include/kvp.h declares."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2508_13231_b200 import build
    return ctypes.CDLL(build.build_library())


def _declared():
    text = open(os.path.join(ROOT, "include", "kvp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvp_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    from paper_2508_13231_b200 import kvp
    assert sorted(kvp.EXPORTS) == names


def test_host_only_entry_points(lib, oracle):
    # Philox and the acceptance table are pure host code: they must agree with the oracle bit for bit
    out = (ctypes.c_uint32 * 4)()
    lib.kvp_philox4x32_10((ctypes.c_uint32 * 4)(1, 2, 3, 4), (ctypes.c_uint32 * 2)(5, 6), out)
    assert tuple(out) == oracle.philox((1, 2, 3, 4), (5, 6))
    temps = np.array([1e9, 31337.5, 800.0, 17.25, 1.0, 0.3], np.float64)
    table = np.zeros((temps.size, 1024), np.uint32)
    shifts = np.zeros(temps.size, np.uint32)
    rc = lib.kvp_accept_table(temps.ctypes.data_as(ctypes.c_void_p), ctypes.c_uint32(temps.size),
                              table.ctypes.data_as(ctypes.c_void_p), shifts.ctypes.data_as(ctypes.c_void_p))
    assert rc == 0
    otable, oshifts = oracle.accept_table(temps)
    assert np.array_equal(table, otable) and np.array_equal(shifts, oshifts)
    # long ladders are built by several host threads, rows split unevenly when the level count is no multiple
    # (equal neighbours, as in a ladder that has cooled below one tick, share a row: the last case has runs of them
    # at the start, in the middle and at the end)
    ladders = [c0 * alpha ** np.arange(levels, dtype=np.float64)
               for levels, c0, alpha in ((64, 54321.0, 0.9), (100, 7.5e6, 0.83), (17, 3.0, 0.5))]
    ladders.append(np.array([5.0, 5.0, 0.2, 0.1, 9.0] + [700.0] * 20 + [9.0, 9.0, 0.5, 0.5], np.float64))
    for temps in ladders:
        levels = temps.size
        table = np.zeros((levels, 1024), np.uint32)
        shifts = np.zeros(levels, np.uint32)
        assert lib.kvp_accept_table(temps.ctypes.data_as(ctypes.c_void_p), ctypes.c_uint32(levels),
                                    table.ctypes.data_as(ctypes.c_void_p), shifts.ctypes.data_as(ctypes.c_void_p)) == 0
        otable, oshifts = oracle.accept_table(temps)
        assert np.array_equal(table, otable) and np.array_equal(shifts, oshifts)
    lib.kvp_strerror.restype = ctypes.c_char_p
    assert lib.kvp_strerror(0) == b"ok" and b"capacity" in lib.kvp_strerror(-2)
    assert lib.kvp_accept_table(None, 1, None, None) == -1


def test_no_gpu_means_error_not_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    class MemSys(ctypes.Structure):
        _fields_ = [("a", ctypes.c_uint64), ("b", ctypes.c_uint64), ("c", ctypes.c_uint64),
                    ("f", ctypes.c_uint32), ("r", ctypes.c_uint32)]
    h = ctypes.c_void_p()
    ms = MemSys(8, 1, 1, 3, 0)
    dummy = np.zeros(4, np.uint32)
    rc = lib.kvp_create(ctypes.byref(h), 16, ctypes.c_uint64(8192), 4, dummy.ctypes.data_as(ctypes.c_void_p), 4,
                        ctypes.byref(ms), None, None, None)
    assert rc in (-4, -5)      # KVP_ERR_CUDA: no device, and no CPU path to fall back to

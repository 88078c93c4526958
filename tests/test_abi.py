"""The C-ABI library loads, exports every declared symbol and validates its
arguments on the host before touching a GPU.  No GPU needed."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2411_02581_b200 import binding as B
from paper_2411_02581_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tuna.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tuna_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
        assert n in B.SIGNATURES, n
    assert sorted(B.SIGNATURES) == names


def test_version_and_strerror(lib):
    assert lib.tuna_version() >= 100
    for code in range(0, -11, -1):
        s = lib.tuna_strerror(code)
        assert s and s != b"unknown status"
    assert lib.tuna_strerror(-99) == b"unknown status"


def _create(lib, P, radix, rg, l, g, elem, counts, sdispls=None):
    h = ctypes.c_void_p()
    c = np.ascontiguousarray(counts, dtype=np.int64)
    cp = c.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))
    sp = None
    if sdispls is not None:
        s = np.ascontiguousarray(sdispls, dtype=np.int64)
        sp = s.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))
    rc = lib.tuna_plan_create(ctypes.byref(h), P, radix, rg, l, g, elem, 0, cp, sp, None, None,
                              None, None)
    assert not h.value or rc == 0
    return rc


def test_host_validation_rejects_before_any_gpu_work(lib):
    z = np.zeros((4, 4), dtype=np.int64)
    assert _create(lib, 0, 2, 2, 1, 1, 1, z) == -1            # P < 1
    assert _create(lib, 4, 2, 2, 4, 1, 0, z) == -1            # elem_size < 1
    assert _create(lib, 4, 2, 2, 3, 2, 1, z) == -3            # l * g != P
    assert _create(lib, 4, 1, 2, 4, 1, 1, z) == -2            # radix < 2
    assert _create(lib, 4, 5, 2, 4, 1, 1, z) == -2            # radix > P
    assert _create(lib, 4, 2, 3, 2, 2, 1, z) == -2            # global radix > g
    neg = z.copy()
    neg[1, 2] = -1
    assert _create(lib, 4, 2, 2, 4, 1, 1, neg) == -1          # negative count
    assert _create(lib, 4, 2, 2, 4, 1, 1, z, sdispls=neg) == -1
    assert lib.tuna_plan_create(None, 4, 2, 2, 4, 1, 1, 0, None, None, None, None, None, None) == -1
    assert lib.tuna_plan_destroy(None) == 0
    n = ctypes.c_size_t()
    assert lib.tuna_plan_workspace_bytes(None, ctypes.byref(n)) == -1
    assert lib.tuna_alltoallv(None, None, None, None, None, None, None, None) == -1


def test_radix_zero_means_choose_and_rank_limit(lib):
    z = np.zeros((4, 4), dtype=np.int64)
    # radix 0 passes validation (what follows needs a GPU: without one the first CUDA
    # call fails, with one the plan is built); it is not a radix error either way
    assert _create(lib, 4, 0, 0, 2, 2, 1, z) in (0, -7, -8)
    assert _create(lib, 4, 0, 2, 4, 1, 1, z) in (0, -7, -8)
    big = np.zeros((1, 1), dtype=np.int64)
    assert _create(lib, 32769, 2, 2, 32769, 1, 1, big) == -9   # above TUNA_MAX_P: refused before the counts are read


def _static(lib, P, elem, counts, sdispls=None, sendbase=None):
    def arr(a):
        if a is None:
            return None, None
        a = np.ascontiguousarray(a, dtype=np.int64)
        return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))
    c, cp = arr(counts)
    s, sp = arr(sdispls)
    b, bp = arr(sendbase)
    return lib.tuna_direct_alltoallv_static(P, elem, cp, sp, None, bp, None, None, None, None)


def test_static_entry_refuses_sizes_before_it_looks_at_buffers(lib):
    """Limits of the allocation-free entry point, with NULL buffers and no GPU: a size
    over a limit must come back as TUNA_ERR_RANGE, never reach a launch."""
    huge = np.zeros((2, 2), dtype=np.int64)
    huge[0, 1] = 5 << 30                                       # 5 GiB of blocks: work stream over 4 GiB
    assert _static(lib, 2, 1, huge) == -9
    many = np.full((2, 2), 1 << 30, dtype=np.int64)            # 4 x 1 Gi elements of 8 bytes
    assert _static(lib, 2, 8, many) == -9
    wrap = np.zeros((2, 2), dtype=np.int64)
    wrap[1, 0] = (1 << 62) // 3                                # bytes = count * 12 would wrap
    assert _static(lib, 2, 12, wrap) == -9
    small = np.ones((2, 2), dtype=np.int64)
    far = np.zeros((2, 2), dtype=np.int64)
    far[0, 0] = 1 << 60                                        # displacement + count beyond any buffer
    assert _static(lib, 2, 1, small, sdispls=far) == -9
    assert _static(lib, 2, 1, small, sendbase=[0, 1 << 61]) == -9
    assert _static(lib, 129, 1, np.zeros((129, 129), dtype=np.int64)) == -9     # above TUNA_STATIC_MAX_P
    assert _static(lib, 2, 1, small) == -1                     # fine sizes, NULL buffers
    neg = small.copy()
    neg[0, 1] = -1
    assert _static(lib, 2, 1, neg) == -1


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(build_mod, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.lib()

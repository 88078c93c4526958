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


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(build_mod, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.lib()

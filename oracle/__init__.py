"""ctypes front end of the CPU oracle (``tuna_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package.  The C file is compiled with gcc on first use.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tuna_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB = os.path.join(_OUT_DIR, "libtuna_oracle.so")
# The mutation tests point this at a deliberately broken copy of the source to
# check that the pins notice; nothing else sets it.
if os.environ.get("TUNA_ORACLE_SOURCE"):
    _SRC = os.environ["TUNA_ORACLE_SOURCE"]
    _OUT_DIR = os.path.dirname(_SRC)
    _LIB = os.path.splitext(_SRC)[0] + ".so"
_SRC_MT = os.path.join(_HERE, "tuna_oracle_mt.c")       # threaded timing variant (not the checker)
_LIB_MT = os.path.join(_HERE, "_build", "libtuna_oracle_mt.so")
_lock = threading.Lock()
_lib = None
_lib_mt = None

RS_COLS = 6
RS_LEVEL, RS_X, RS_Z, RS_UNITS, RS_BYTES_SENT, RS_BYTES_RECV = range(6)
TR_COLS = 8
TR_ROUND, TR_KIND, TR_PARTNER, TR_OFFSET, TR_ORIGIN, TR_DEST, TR_BYTES, TR_PLACE = range(8)


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object beside its source."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def build_mt(force: bool = False) -> str:
    """Compile the threaded timing variant of the flat oracle."""
    os.makedirs(os.path.dirname(_LIB_MT), exist_ok=True)
    if force or not os.path.exists(_LIB_MT) or os.path.getmtime(_LIB_MT) < os.path.getmtime(_SRC_MT):
        tmp = _LIB_MT + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=gnu11", "-Wall", "-Wextra", "-shared", "-fPIC", "-pthread",
                               "-o", tmp, _SRC_MT])
        os.replace(tmp, _LIB_MT)
    return _LIB_MT


_I64P = ctypes.POINTER(ctypes.c_int64)
_U8P = ctypes.POINTER(ctypes.c_uint8)
_IP = ctypes.POINTER(ctypes.c_int)


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.oracle_num_digits.argtypes = [ctypes.c_int, ctypes.c_int]
            lib.oracle_round_list.argtypes = [ctypes.c_int, ctypes.c_int, _IP, _IP, ctypes.c_int]
            lib.oracle_tmap.argtypes = [ctypes.c_int] * 3
            lib.oracle_bruteforce.argtypes = [ctypes.c_int, ctypes.c_int] + [_I64P] * 5 + [_U8P, _U8P]
            lib.oracle_tuna_flat.argtypes = (
                [ctypes.c_int] * 3 + [_I64P] * 5 + [_U8P, _U8P, _I64P, ctypes.c_int, _IP, _IP,
                                                    ctypes.c_int, _I64P, ctypes.c_int64, _I64P,
                                                    _I64P])
            lib.oracle_segmented_exclusive_scan.argtypes = [_I64P, ctypes.c_int64, ctypes.c_int64,
                                                            ctypes.c_int64, _I64P, _I64P]
            lib.oracle_tuna_hier.argtypes = (
                [ctypes.c_int] * 5 + [_I64P] * 5 + [_U8P, _U8P, ctypes.c_int64, _U8P, _I64P,
                                                    ctypes.c_int, _IP])
            lib.oracle_tuna_hier_tables.argtypes = (
                [ctypes.c_int] * 5 + [_I64P] * 5 + [_U8P, _U8P, ctypes.c_int64, _U8P, _I64P, _I64P,
                                                    _I64P])
            lib.oracle_tuna_hier_staggered.argtypes = (
                [ctypes.c_int] * 5 + [_I64P] * 5 + [_U8P, _U8P, ctypes.c_int64, _U8P, _I64P,
                                                    ctypes.c_int, _IP, _IP])
            lib.oracle_rows_alltoallv.argtypes = ([ctypes.c_int, ctypes.c_int64] + [_I64P] * 7
                                                  + [_U8P, ctypes.c_int64, _U8P, ctypes.c_int64])
            _lib = lib
    return _lib


def _i64(a):
    a = np.ascontiguousarray(a, dtype=np.int64)
    return a, a.ctypes.data_as(_I64P)


def _u8(a):
    assert a.dtype == np.uint8 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_U8P)


def num_digits(P: int, r: int) -> int:
    return _load().oracle_num_digits(P, r)


def round_list(P: int, r: int):
    """The rounds [(x, z), ...] of a flat exchange in execution order."""
    lib = _load()
    K = lib.oracle_round_list(P, r, None, None, 0)
    xs = (ctypes.c_int * max(K, 1))()
    zs = (ctypes.c_int * max(K, 1))()
    lib.oracle_round_list(P, r, xs, zs, K)
    return [(xs[i], zs[i]) for i in range(K)]


def tmap(P: int, r: int, o: int) -> int:
    return _load().oracle_tmap(P, r, o)


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"{what} failed with oracle status {rc}")


def bruteforce(wl, send: np.ndarray, recv: np.ndarray) -> np.ndarray:
    """The exchange by its definition; writes into and returns ``recv``."""
    c, cp = _i64(wl.sendcounts)
    sd, sdp = _i64(wl.sdispls)
    rd, rdp = _i64(wl.rdispls)
    sb, sbp = _i64(wl.sendbase)
    rb, rbp = _i64(wl.recvbase)
    _check(_load().oracle_bruteforce(wl.P, wl.elem_size, cp, sdp, rdp, sbp, rbp, _u8(send),
                                     _u8(recv)), "oracle_bruteforce")
    return recv


def segmented_exclusive_scan(val: np.ndarray, align: int = 1):
    """Per-row exclusive running sums of a 2-D int64 array; returns (scan, row totals)."""
    v, vp = _i64(val)
    nseg, seglen = v.shape
    out = np.zeros_like(v)
    tot = np.zeros(nseg, dtype=np.int64)
    _check(_load().oracle_segmented_exclusive_scan(vp, nseg, seglen, align,
                                                   out.ctypes.data_as(_I64P),
                                                   tot.ctypes.data_as(_I64P)),
           "oracle_segmented_exclusive_scan")
    return out, tot


def tuna_flat(wl, r: int, send: np.ndarray, recv: np.ndarray, trace_rank: int = -1,
              want_sizes: bool = False):
    """Algorithm 1.  Returns (recv, rounds[K, RS_COLS], B, trace or None); with
    ``want_sizes`` a fifth item: the size tables [w, P, P] after every digit phase."""
    lib = _load()
    c, cp = _i64(wl.sendcounts)
    sd, sdp = _i64(wl.sdispls)
    rd, rdp = _i64(wl.rdispls)
    sb, sbp = _i64(wl.sendbase)
    rb, rbp = _i64(wl.recvbase)
    K = lib.oracle_round_list(wl.P, r, None, None, 0)
    rounds = np.zeros((max(K, 1), RS_COLS), dtype=np.int64)
    Kc, Bc = ctypes.c_int(0), ctypes.c_int(0)
    trace = None
    tp, tcap, trows = None, 0, ctypes.c_int64(0)
    if trace_rank >= 0:
        tcap = 2 * wl.P * max(K, 1)
        trace = np.zeros((tcap, TR_COLS), dtype=np.int64)
        tp = trace.ctypes.data_as(_I64P)
    sizes, szp = None, None
    if want_sizes:
        sizes = np.zeros((max(lib.oracle_num_digits(wl.P, r), 1), wl.P, wl.P), dtype=np.int64)
        szp = sizes.ctypes.data_as(_I64P)
    _check(lib.oracle_tuna_flat(wl.P, r, wl.elem_size, cp, sdp, rdp, sbp, rbp, _u8(send),
                                _u8(recv), rounds.ctypes.data_as(_I64P), K, ctypes.byref(Kc),
                                ctypes.byref(Bc), trace_rank, tp, tcap, ctypes.byref(trows), szp),
           "oracle_tuna_flat")
    assert Kc.value == K
    if trace is not None:
        assert trows.value <= tcap
        trace = trace[:trows.value]
    if want_sizes:
        return recv, rounds[:K], Bc.value, trace, sizes[:lib.oracle_num_digits(wl.P, r)]
    return recv, rounds[:K], Bc.value, trace


def tuna_flat_mt(wl, r: int, send: np.ndarray, recv: np.ndarray, threads: int):
    """Algorithm 1 with the ranks of every round shared out over ``threads`` plain threads:
    a TIMING variant for the CPU baseline, checked against :func:`tuna_flat` by a test; never
    used to check anything itself.  Returns (recv, rounds[K, RS_COLS])."""
    global _lib_mt
    with _lock:
        if _lib_mt is None:
            lib = ctypes.CDLL(build_mt())
            lib.oracle_tuna_flat_mt.argtypes = ([ctypes.c_int] * 3 + [_I64P] * 5
                                                + [_U8P, _U8P, _I64P, ctypes.c_int, ctypes.c_int])
            _lib_mt = lib
    c, cp = _i64(wl.sendcounts)
    sd, sdp = _i64(wl.sdispls)
    rd, rdp = _i64(wl.rdispls)
    sb, sbp = _i64(wl.sendbase)
    rb, rbp = _i64(wl.recvbase)
    K = _load().oracle_round_list(wl.P, r, None, None, 0)
    rounds = np.zeros((max(K, 1), RS_COLS), dtype=np.int64)
    _check(_lib_mt.oracle_tuna_flat_mt(wl.P, r, wl.elem_size, cp, sdp, rdp, sbp, rbp, _u8(send),
                                       _u8(recv), rounds.ctypes.data_as(_I64P), K, int(threads)),
           "oracle_tuna_flat_mt")
    return recv, rounds[:K]


def tuna_hier(wl, Q: int, N: int, rl: int, rg: int, send: np.ndarray, recv: np.ndarray,
              want_after_local: bool = False):
    """Hierarchical exchange.  Returns (recv, rounds, (K_local, K_global), recv_after_local)."""
    lib = _load()
    assert Q * N == wl.P
    c, cp = _i64(wl.sendcounts)
    sd, sdp = _i64(wl.sdispls)
    rd, rdp = _i64(wl.rdispls)
    sb, sbp = _i64(wl.sendbase)
    rb, rbp = _i64(wl.recvbase)
    K = lib.oracle_round_list(Q, rl, None, None, 0) + lib.oracle_round_list(N, rg, None, None, 0)
    rounds = np.zeros((max(K, 1), RS_COLS), dtype=np.int64)
    Ks = (ctypes.c_int * 2)()
    after = np.empty_like(recv) if want_after_local else None
    _check(lib.oracle_tuna_hier(Q, N, rl, rg, wl.elem_size, cp, sdp, rdp, sbp, rbp, _u8(send),
                                _u8(recv), recv.nbytes, _u8(after) if after is not None else None,
                                rounds.ctypes.data_as(_I64P), K, Ks), "oracle_tuna_hier")
    assert Ks[0] + Ks[1] == K
    return recv, rounds[:K], (Ks[0], Ks[1]), after


def tuna_hier_tables(wl, Q: int, N: int, rl: int, rg: int, send: np.ndarray, recv: np.ndarray):
    """The hierarchical exchange with the metadata the ranks hold copied out.  Returns
    (recv, recv_after_local, sz_local[wl, P, N, Q], usz_compact[P, N, Q],
    usz_global[wg, P, N, Q]): block sizes by (rank, destination group, local offset) after
    every local digit phase; sub-block sizes by (rank, group offset, source local id) after
    the compaction and after every global digit phase."""
    lib = _load()
    assert Q * N == wl.P
    P = wl.P
    c, cp = _i64(wl.sendcounts)
    sd, sdp = _i64(wl.sdispls)
    rd, rdp = _i64(wl.rdispls)
    sb, sbp = _i64(wl.sendbase)
    rb, rbp = _i64(wl.recvbase)
    wloc, wglo = lib.oracle_num_digits(Q, rl), lib.oracle_num_digits(N, rg)
    sz_local = np.zeros((max(wloc, 1), P, N, Q), dtype=np.int64)
    usz_compact = np.zeros((P, N, Q), dtype=np.int64)
    usz_global = np.zeros((max(wglo, 1), P, N, Q), dtype=np.int64)
    after = np.empty_like(recv)
    _check(lib.oracle_tuna_hier_tables(Q, N, rl, rg, wl.elem_size, cp, sdp, rdp, sbp, rbp, _u8(send),
                                       _u8(recv), recv.nbytes, _u8(after),
                                       sz_local.ctypes.data_as(_I64P),
                                       usz_compact.ctypes.data_as(_I64P),
                                       usz_global.ctypes.data_as(_I64P)), "oracle_tuna_hier_tables")
    return recv, after, sz_local[:wloc], usz_compact, usz_global[:wglo]


def tuna_hier_staggered(wl, Q: int, N: int, rl: int, block_count: int, send: np.ndarray,
                        recv: np.ndarray):
    """Local phase, then the staggered inter-group exchange in batches of ``block_count``
    steps.  Returns (recv, rounds, (K_local, K_global), batches)."""
    lib = _load()
    assert Q * N == wl.P
    c, cp = _i64(wl.sendcounts)
    sd, sdp = _i64(wl.sdispls)
    rd, rdp = _i64(wl.rdispls)
    sb, sbp = _i64(wl.sendbase)
    rb, rbp = _i64(wl.recvbase)
    K = lib.oracle_round_list(Q, rl, None, None, 0) + Q * (N - 1)
    rounds = np.zeros((max(K, 1), RS_COLS), dtype=np.int64)
    Ks = (ctypes.c_int * 2)()
    batches = ctypes.c_int(0)
    _check(lib.oracle_tuna_hier_staggered(Q, N, rl, block_count, wl.elem_size, cp, sdp, rdp, sbp,
                                          rbp, _u8(send), _u8(recv), recv.nbytes, None,
                                          rounds.ctypes.data_as(_I64P), K, Ks,
                                          ctypes.byref(batches)), "oracle_tuna_hier_staggered")
    assert Ks[0] + Ks[1] == K
    return recv, rounds[:K], (Ks[0], Ks[1]), batches.value


def rows_alltoallv(wl, gather, scatter, rows_in: np.ndarray, rows_out: np.ndarray) -> np.ndarray:
    """Exchange of whole rows with a gather in front and a scatter behind (not in the
    paper).  ``wl`` counts rows of ``wl.elem_size`` bytes; ``rows_in`` / ``rows_out`` are
    2-D uint8 arrays [rows, elem_size]; ``gather`` / ``scatter`` are int64 row maps or None."""
    lib = _load()
    c, cp = _i64(wl.sendcounts)
    sd, sdp = _i64(wl.sdispls)
    rd, rdp = _i64(wl.rdispls)
    sb, sbp = _i64(wl.sendbase)
    rb, rbp = _i64(wl.recvbase)
    g = gp = s = sp = None
    if gather is not None:
        g, gp = _i64(gather)
    if scatter is not None:
        s, sp = _i64(scatter)
    assert rows_in.shape[1] == rows_out.shape[1] == wl.elem_size
    _check(lib.oracle_rows_alltoallv(wl.P, wl.elem_size, cp, sdp, rdp, sbp, rbp, gp, sp, _u8(rows_in),
                                     rows_in.shape[0], _u8(rows_out), rows_out.shape[0]),
           "oracle_rows_alltoallv")
    return rows_out

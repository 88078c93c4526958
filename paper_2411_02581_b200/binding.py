"""Thin ctypes binding over the C ABI declared in ``include/tuna.h``.

Only argument marshalling happens here: every step of the exchange runs in the
CUDA library.  There is no CPU fallback; if the shared library is missing the
import of :func:`lib` raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from . import build as _build

_I64P = ctypes.POINTER(ctypes.c_int64)
_INTP = ctypes.POINTER(ctypes.c_int)
_SZP = ctypes.POINTER(ctypes.c_size_t)
_VP = ctypes.c_void_p

FLAG_DIRECT_TO_R = 0
FLAG_CLASSIC_ROTATE = 1
FLAG_BULK_COPY = 2
FLAG_NO_DIRECT = 4
PART_KEEP = 0
PART_DELIVER = 1
SHARD_LOCAL = 1
SHARD_GLOBAL = 2
SCHEDULE_TUNA = 0
SCHEDULE_DIRECT = 1
HOST_STAGED = 0x100

TIMER_NAMES = ("plan", "round_local", "round_global", "rotate", "direct")
TIMER_KINDS = len(TIMER_NAMES)

STATUS = {
    0: "TUNA_OK", -1: "TUNA_ERR_INVALID_ARG", -2: "TUNA_ERR_BAD_RADIX",
    -3: "TUNA_ERR_BAD_HIERARCHY", -4: "TUNA_ERR_COUNT_MISMATCH", -5: "TUNA_ERR_OVERLAP",
    -6: "TUNA_ERR_WORKSPACE", -7: "TUNA_ERR_CUDA", -8: "TUNA_ERR_NOMEM", -9: "TUNA_ERR_RANGE", -10: "TUNA_ERR_INTERNAL",
}

# name -> (restype, argtypes); must list every symbol include/tuna.h declares
SIGNATURES = {
    "tuna_plan_create": (ctypes.c_int, [ctypes.POINTER(_VP)] + [ctypes.c_int] * 6 + [ctypes.c_uint]
                         + [_I64P] * 5 + [_VP]),
    "tuna_plan_create_staggered": (ctypes.c_int, [ctypes.POINTER(_VP)] + [ctypes.c_int] * 6
                                   + [ctypes.c_uint] + [_I64P] * 5 + [_VP]),
    "tuna_plan_update_counts": (ctypes.c_int, [_VP] + [_I64P] * 5 + [_VP]),
    "tuna_plan_update_counts_device": (ctypes.c_int, [_VP, _VP, _VP]),
    "tuna_plan_set_row_maps": (ctypes.c_int, [_VP, _VP, _VP, ctypes.c_int64, ctypes.c_int64, _VP]),
    "tuna_rows_alltoallv": (ctypes.c_int, [_VP, _VP, _VP, _VP]),
    "tuna_plan_destroy": (ctypes.c_int, [_VP]),
    "tuna_plan_workspace_bytes": (ctypes.c_int, [_VP, _SZP]),
    "tuna_plan_host_staging_bytes": (ctypes.c_int, [_VP, _SZP]),
    "tuna_plan_set_workspace": (ctypes.c_int, [_VP, _VP, ctypes.c_size_t]),
    "tuna_plan_extents": (ctypes.c_int, [_VP, _SZP, _SZP, _SZP]),
    "tuna_alltoallv": (ctypes.c_int, [_VP, _VP, _I64P, _I64P, _VP, _I64P, _I64P, _VP]),
    "tuna_direct_alltoallv": (ctypes.c_int, [_VP, _VP, _I64P, _I64P, _VP, _I64P, _I64P, _VP]),
    "tuna_alltoallv_host": (ctypes.c_int, [_VP, _VP, _VP, ctypes.c_int, _VP]),
    "tuna_direct_alltoallv_static": (ctypes.c_int, [ctypes.c_int, ctypes.c_int] + [_I64P] * 5 + [_VP, _VP, _VP]),
    "tuna_shard_plan_create": (ctypes.c_int, [ctypes.POINTER(_VP)] + [ctypes.c_int] * 5 + [ctypes.c_uint]
                               + [_I64P] * 5 + [_VP]),
    "tuna_shard_extents": (ctypes.c_int, [_VP, ctypes.c_int, _SZP, _SZP]),
    "tuna_shard_layout": (ctypes.c_int, [ctypes.c_int] * 3 + [_I64P] * 9),
    "tuna_shard_round_table": (ctypes.c_int, [ctypes.c_int] * 5 + [_I64P, ctypes.c_int, _INTP, _INTP, _INTP,
                                                                _I64P, _I64P, _INTP]),
    "tuna_shard_enable_peer_access": (ctypes.c_int, [ctypes.c_int]),
    "tuna_shard_alltoallv": (ctypes.c_int, [_VP, _VP, ctypes.POINTER(_VP), ctypes.c_int, _VP]),
    "tuna_plan_num_rounds": (ctypes.c_int, [_VP, _INTP]),
    "tuna_plan_round_info": (ctypes.c_int, [_VP, ctypes.c_int, _INTP, _INTP, _INTP, _I64P, _I64P]),
    "tuna_plan_num_phases": (ctypes.c_int, [_VP, _INTP]),
    "tuna_plan_phase_info": (ctypes.c_int, [_VP, ctypes.c_int, ctypes.c_int, _INTP, _INTP, _I64P, _I64P, _I64P]),
    "tuna_plan_phase_tables": (ctypes.c_int, [_VP, ctypes.c_int, ctypes.c_int, ctypes.c_int64] + [_I64P] * 5),
    "tuna_plan_last_launches": (ctypes.c_int, [_VP, _INTP]),
    "tuna_plan_last_small_launches": (ctypes.c_int, [_VP, _INTP]),
    "tuna_plan_launch_count": (ctypes.c_int, [_VP, _I64P]),
    "tuna_plan_enable_timing": (ctypes.c_int, [_VP, ctypes.c_int]),
    "tuna_plan_get_timing": (ctypes.c_int, [_VP, ctypes.c_int, ctypes.POINTER(ctypes.c_double), _I64P, _I64P]),
    "tuna_plan_cuda_error": (ctypes.c_int, [_VP]),
    "tuna_plan_device_status": (ctypes.c_int, [_VP, _INTP]),
    "tuna_strerror": (ctypes.c_char_p, [ctypes.c_int]),
    "tuna_version": (ctypes.c_int, []),
}

_lib = None


class TunaError(RuntimeError):
    def __init__(self, status: int, what: str, cuda: int = 0):
        self.status = status
        self.cuda_error = cuda
        super().__init__(f"{what}: {STATUS.get(status, status)}"
                         + (f" (cudaError {cuda})" if cuda else ""))


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built in-tree); raise if it does not exist."""
    global _lib
    if _lib is None:
        path = os.environ.get("TUNA_LIBRARY") or _build.LIB_PATH  # override: another build of the library
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build it with `python -m paper_2411_02581_b200.build` "
                "(there is no CPU fallback)")
        l = ctypes.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype = res
            fn.argtypes = args
        _lib = l
    return _lib


def _h(a):
    """Host int64 array (or None) -> (keepalive, pointer)."""
    if a is None:
        return None, None
    a = np.ascontiguousarray(a, dtype=np.int64)
    return a, a.ctypes.data_as(_I64P)


def _ptr(t):
    """Device/host pointer of a torch tensor, numpy array or int."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class Plan:
    """Owner of a ``tuna_plan_t``; methods carry the C function names."""

    def __init__(self, P, radix, l=None, g=1, radix_global=2, elem_size=1, flags=0,
                 sendcounts=None, sdispls=None, rdispls=None, sendbase=None, recvbase=None,
                 stream=None, block_count=0, shard=None):
        """``block_count`` > 0 selects ``tuna_plan_create_staggered`` (``radix_global`` unused);
        ``shard`` = (n_gpus, my_gpu) selects ``tuna_shard_plan_create`` (``l``, ``g`` unused)."""
        self._h = _VP()
        self._ws = None
        l = P if l is None else l
        keep = [_h(x) for x in (sendcounts, sdispls, rdispls, sendbase, recvbase)]
        if shard is not None:
            what = "tuna_shard_plan_create"
            rc = lib().tuna_shard_plan_create(ctypes.byref(self._h), P, radix, shard[0], shard[1],
                                              elem_size, flags, *[k[1] for k in keep], _stream(stream))
        elif block_count:
            what = "tuna_plan_create_staggered"
            rc = lib().tuna_plan_create_staggered(ctypes.byref(self._h), P, radix, block_count, l, g,
                                                  elem_size, flags, *[k[1] for k in keep],
                                                  _stream(stream))
        else:
            what = "tuna_plan_create"
            rc = lib().tuna_plan_create(ctypes.byref(self._h), P, radix, radix_global, l, g,
                                        elem_size, flags, *[k[1] for k in keep], _stream(stream))
        if rc != 0:
            self._h = _VP()
            raise TunaError(rc, what)
        self.P, self.elem_size = P, elem_size

    def _check(self, rc, what):
        if rc != 0:
            raise TunaError(rc, what, lib().tuna_plan_cuda_error(self._h))

    def destroy(self):
        if self._h:
            lib().tuna_plan_destroy(self._h)
            self._h = _VP()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def update_counts(self, sendcounts, sdispls=None, rdispls=None, sendbase=None, recvbase=None,
                      stream=None):
        keep = [_h(x) for x in (sendcounts, sdispls, rdispls, sendbase, recvbase)]
        self._check(lib().tuna_plan_update_counts(self._h, *[k[1] for k in keep], _stream(stream)),
                    "tuna_plan_update_counts")

    def update_counts_device(self, d_sendcounts, stream=None):
        """New counts from a P x P int64 array in device memory (packed layout)."""
        self._check(lib().tuna_plan_update_counts_device(self._h, _ptr(d_sendcounts), _stream(stream)),
                    "tuna_plan_update_counts_device")

    def workspace_bytes(self) -> int:
        n = ctypes.c_size_t()
        self._check(lib().tuna_plan_workspace_bytes(self._h, ctypes.byref(n)), "tuna_plan_workspace_bytes")
        return n.value

    def host_staging_bytes(self) -> int:
        n = ctypes.c_size_t()
        self._check(lib().tuna_plan_host_staging_bytes(self._h, ctypes.byref(n)),
                    "tuna_plan_host_staging_bytes")
        return n.value

    def set_workspace(self, tensor, nbytes=None):
        """``tensor``: a torch uint8 CUDA tensor (kept alive by the plan) or None."""
        self._ws = tensor
        nb = 0 if tensor is None else (tensor.numel() * tensor.element_size() if nbytes is None else nbytes)
        self._check(lib().tuna_plan_set_workspace(self._h, _ptr(tensor), nb), "tuna_plan_set_workspace")

    def alloc_workspace(self, host_staging=False, device="cuda"):
        """Allocate the workspace through torch (256-byte aligned) and attach it."""
        import torch
        need = self.workspace_bytes()
        need = (need + 255) // 256 * 256 + (self.host_staging_bytes() if host_staging else 0)
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=device)
        self.set_workspace(ws)
        return ws

    def extents(self):
        a, b, c = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
        self._check(lib().tuna_plan_extents(self._h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
                    "tuna_plan_extents")
        return a.value, b.value, c.value

    def alltoallv(self, sendbuf, recvbuf, sendcounts=None, sdispls=None, recvcounts=None,
                  rdispls=None, stream=None):
        keep = [_h(x) for x in (sendcounts, sdispls, recvcounts, rdispls)]
        self._check(lib().tuna_alltoallv(self._h, _ptr(sendbuf), keep[0][1], keep[1][1],
                                         _ptr(recvbuf), keep[2][1], keep[3][1], _stream(stream)),
                    "tuna_alltoallv")

    def direct_alltoallv(self, sendbuf, recvbuf, sendcounts=None, sdispls=None, recvcounts=None,
                         rdispls=None, stream=None):
        keep = [_h(x) for x in (sendcounts, sdispls, recvcounts, rdispls)]
        self._check(lib().tuna_direct_alltoallv(self._h, _ptr(sendbuf), keep[0][1], keep[1][1],
                                                _ptr(recvbuf), keep[2][1], keep[3][1],
                                                _stream(stream)), "tuna_direct_alltoallv")

    def set_row_maps(self, gather_rows, scatter_rows, in_rows: int, out_rows: int, stream=None):
        """``gather_rows`` / ``scatter_rows``: int64 CUDA tensors or None (identity)."""
        self._check(lib().tuna_plan_set_row_maps(
            self._h, _ptr(gather_rows) if gather_rows is not None else None,
            _ptr(scatter_rows) if scatter_rows is not None else None, in_rows, out_rows,
            _stream(stream)), "tuna_plan_set_row_maps")

    def rows_alltoallv(self, rows_in, rows_out, stream=None):
        self._check(lib().tuna_rows_alltoallv(self._h, _ptr(rows_in), _ptr(rows_out), _stream(stream)),
                    "tuna_rows_alltoallv")

    def shard_extents(self, gpu):
        a, b = ctypes.c_size_t(), ctypes.c_size_t()
        self._check(lib().tuna_shard_extents(self._h, gpu, ctypes.byref(a), ctypes.byref(b)),
                    "tuna_shard_extents")
        return a.value, b.value

    def shard_alltoallv(self, sendbuf, recvbufs, phases=SHARD_LOCAL | SHARD_GLOBAL, stream=None):
        """``recvbufs``: one tensor (or address) per GPU, as this process addresses them."""
        ptrs = (_VP * len(recvbufs))(*[_ptr(r) for r in recvbufs])
        self._check(lib().tuna_shard_alltoallv(self._h, _ptr(sendbuf), ptrs, phases, _stream(stream)),
                    "tuna_shard_alltoallv")

    def alltoallv_host(self, host_send, host_recv, schedule=SCHEDULE_TUNA, stream=None):
        self._check(lib().tuna_alltoallv_host(self._h, _ptr(host_send), _ptr(host_recv), schedule,
                                              _stream(stream)), "tuna_alltoallv_host")

    def num_rounds(self) -> int:
        k = ctypes.c_int()
        self._check(lib().tuna_plan_num_rounds(self._h, ctypes.byref(k)), "tuna_plan_num_rounds")
        return k.value

    def round_info(self, k):
        lv, x, z = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        u, b = ctypes.c_int64(), ctypes.c_int64()
        self._check(lib().tuna_plan_round_info(self._h, k, ctypes.byref(lv), ctypes.byref(x),
                                               ctypes.byref(z), ctypes.byref(u), ctypes.byref(b)),
                    "tuna_plan_round_info")
        return dict(level=lv.value, x=x.value, z=z.value, units=u.value, bytes=b.value)

    def rounds(self):
        return [self.round_info(k) for k in range(self.num_rounds())]

    def num_phases(self) -> int:
        n = ctypes.c_int()
        self._check(lib().tuna_plan_num_phases(self._h, ctypes.byref(n)), "tuna_plan_num_phases")
        return n.value

    def phase_info(self, phase, part=PART_KEEP):
        lv, x = ctypes.c_int(), ctypes.c_int()
        e, b, s = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
        self._check(lib().tuna_plan_phase_info(self._h, phase, part, ctypes.byref(lv), ctypes.byref(x),
                                               ctypes.byref(e), ctypes.byref(b), ctypes.byref(s)),
                    "tuna_plan_phase_info")
        return dict(level=lv.value, x=x.value, entries=e.value, bytes=b.value, stream_bytes=s.value)

    def phase_tables(self, phase, part=PART_KEEP):
        n = self.phase_info(phase, part)["entries"]
        arrs = [np.zeros(max(n, 1), dtype=np.int64) for _ in range(4)]
        rows = ctypes.c_int64()
        self._check(lib().tuna_plan_phase_tables(self._h, phase, part, n,
                                                 *[a.ctypes.data_as(_I64P) for a in arrs],
                                                 ctypes.byref(rows)), "tuna_plan_phase_tables")
        assert rows.value == n
        return dict(len=arrs[0][:n], pos=arrs[1][:n], src=arrs[2][:n], dst=arrs[3][:n])

    def last_launches(self) -> int:
        n = ctypes.c_int()
        self._check(lib().tuna_plan_last_launches(self._h, ctypes.byref(n)), "tuna_plan_last_launches")
        return n.value
    def last_small_launches(self) -> int:
        n = ctypes.c_int()
        self._check(lib().tuna_plan_last_small_launches(self._h, ctypes.byref(n)),
                    "tuna_plan_last_small_launches")
        return n.value

    def device_status(self) -> int:
        """0, or 1 if a kernel of this plan gave up a bounded wait (synchronises the device)."""
        n = ctypes.c_int()
        self._check(lib().tuna_plan_device_status(self._h, ctypes.byref(n)), "tuna_plan_device_status")
        return n.value

    def launch_count(self) -> int:
        n = ctypes.c_int64()
        self._check(lib().tuna_plan_launch_count(self._h, ctypes.byref(n)), "tuna_plan_launch_count")
        return n.value

    def enable_timing(self, on=True):
        self._check(lib().tuna_plan_enable_timing(self._h, int(bool(on))), "tuna_plan_enable_timing")

    def get_timing(self, reset=True):
        """{kind: dict(ms, launches, bytes)} accumulated since the last reset."""
        ms = (ctypes.c_double * TIMER_KINDS)()
        ln = (ctypes.c_int64 * TIMER_KINDS)()
        by = (ctypes.c_int64 * TIMER_KINDS)()
        self._check(lib().tuna_plan_get_timing(self._h, int(bool(reset)), ms, ln, by), "tuna_plan_get_timing")
        return {name: dict(ms=ms[i], launches=ln[i], bytes=by[i]) for i, name in enumerate(TIMER_NAMES)}


STATIC_MAX_P = 128


def direct_alltoallv_static(P, elem_size, sendcounts, sendbuf, recvbuf, sdispls=None, rdispls=None,
                            sendbase=None, recvbase=None, stream=None):
    """The direct exchange without a plan and without any device allocation: for
    callers whose process may not call cudaMalloc (a framework owns all device
    memory, or allocation is banned inside a latency-critical loop).  Limits: P up
    to STATIC_MAX_P and about 4 GiB of payload; calls must not overlap on the GPU."""
    keep = [_h(x) for x in (sendcounts, sdispls, rdispls, sendbase, recvbase)]
    rc = lib().tuna_direct_alltoallv_static(P, elem_size, *[k[1] for k in keep], _ptr(sendbuf),
                                            _ptr(recvbuf), _stream(stream))
    if rc != 0:
        raise TunaError(rc, "tuna_direct_alltoallv_static")


def shard_layout(P, n_gpus, elem_size, sendcounts, sdispls=None, rdispls=None, sendbase=None,
                 recvbase=None):
    """Host only: (sendbase[P], recvbase[P], send_bytes[n_gpus], recv_bytes[n_gpus]) of a sharded
    layout (``tuna_shard_layout``)."""
    keep = [_h(x) for x in (sendcounts, sdispls, rdispls, sendbase, recvbase)]
    sb, rb = np.zeros(P, dtype=np.int64), np.zeros(P, dtype=np.int64)
    se, re = np.zeros(n_gpus, dtype=np.int64), np.zeros(n_gpus, dtype=np.int64)
    rc = lib().tuna_shard_layout(P, n_gpus, elem_size, *[k[1] for k in keep],
                                 *[a.ctypes.data_as(_I64P) for a in (sb, rb, se, re)])
    if rc != 0:
        raise TunaError(rc, "tuna_shard_layout")
    return sb, rb, se, re


def shard_round_table(P, n_gpus, my_gpu, radix, elem_size, sendcounts):
    """Host only: the rounds of the sharded schedule with what GPU ``my_gpu`` sends in each,
    as a list of dicts like :meth:`Plan.rounds` (``tuna_shard_round_table``)."""
    c, cp = _h(sendcounts)
    n = ctypes.c_int()
    rc = lib().tuna_shard_round_table(P, n_gpus, my_gpu, radix, elem_size, cp, 0, None, None, None, None,
                                      None, ctypes.byref(n))
    if rc != 0:
        raise TunaError(rc, "tuna_shard_round_table")
    K = n.value
    lv, x, z = [(ctypes.c_int * max(K, 1))() for _ in range(3)]
    u, b = np.zeros(max(K, 1), dtype=np.int64), np.zeros(max(K, 1), dtype=np.int64)
    rc = lib().tuna_shard_round_table(P, n_gpus, my_gpu, radix, elem_size, cp, K, lv, x, z,
                                      u.ctypes.data_as(_I64P), b.ctypes.data_as(_I64P), ctypes.byref(n))
    if rc != 0:
        raise TunaError(rc, "tuna_shard_round_table")
    return [dict(level=lv[k], x=x[k], z=z[k], units=int(u[k]), bytes=int(b[k])) for k in range(K)]


def plan_for(wl, radix, l=None, g=1, radix_global=2, flags=0, explicit_layout=True, stream=None,
             block_count=0) -> Plan:
    """A plan for a :class:`workloads.Workload`."""
    kw = dict(sendcounts=wl.sendcounts)
    if explicit_layout:
        kw.update(sdispls=wl.sdispls, rdispls=wl.rdispls, sendbase=wl.sendbase, recvbase=wl.recvbase)
    return Plan(wl.P, radix, l=l, g=g, radix_global=radix_global, elem_size=wl.elem_size,
                flags=flags, stream=stream, block_count=block_count, **kw)

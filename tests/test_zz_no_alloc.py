"""The allocation-free direct exchange against the plan-based one and the CPU oracle.

Some users of this library run where device allocation is off limits: the
framework around them has handed all GPU memory to its own pool, or their
serving loop forbids cudaMalloc after start-up because it stalls every stream.
They call ``tuna_direct_alltoallv_static``, which keeps its tables in a fixed
array inside the library.  This file checks, through the C ABI, that it writes
exactly the bytes ``tuna_direct_alltoallv`` writes, on two calls in a row (the
second one finds the first one's tables in the shared array), and that both
agree with the oracle's definition of the exchange (the two entry points build
their descriptor lists with different code, but a mistake common to both would
pass a comparison between them alone).  It is collected last, so that a run
stopping at the first failure has run everything else.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2411_02581_b200 import binding as B
from paper_2411_02581_b200 import workloads as W

pytestmark = pytest.mark.gpu

CANARY = 0x5C


def plan_based(wl):
    send = wl.make_send("cuda")
    recv = wl.make_recv("cuda", fill=CANARY)
    plan = B.plan_for(wl, 2)
    plan.direct_alltoallv(send, recv)
    torch.cuda.synchronize()
    plan.destroy()
    return send, recv


def no_alloc(wl, send, explicit=True):
    recv = wl.make_recv("cuda", fill=CANARY)
    kw = {}
    if explicit:
        kw = dict(sdispls=wl.sdispls, rdispls=wl.rdispls, sendbase=wl.sendbase, recvbase=wl.recvbase)
    B.direct_alltoallv_static(wl.P, wl.elem_size, wl.sendcounts, send, recv, **kw)
    torch.cuda.synchronize()
    return recv


def test_two_calls_in_a_row_match_the_plan_based_exchange():
    # first call: unaligned byte blocks with gaps; second: a different shape, so
    # that stale tables from the first call would show
    first = W.make_random(37, 900, elem_size=1, seed=41, zero_frac=0.2, gaps=True)
    second = W.make_random(128, 300, elem_size=4, seed=42, zero_frac=0.3)
    for wl, explicit in ((first, True), (second, False), (first, True)):
        send, want = plan_based(wl)
        got = no_alloc(wl, send, explicit)
        assert torch.equal(got, want)            # bit-exact, canaries in the gaps included
        ref = oracle.bruteforce(wl, send.cpu().numpy(), wl.make_recv(fill=CANARY).numpy().copy())
        assert np.array_equal(got.cpu().numpy(), ref)


def test_large_blocks_and_limits():
    wl = W.make_random(4, 3_000_000, elem_size=1, seed=43)
    send, want = plan_based(wl)
    got = no_alloc(wl, send)
    assert torch.equal(got, want)
    ref = oracle.bruteforce(wl, send.cpu().numpy(), wl.make_recv(fill=CANARY).numpy().copy())
    assert np.array_equal(got.cpu().numpy(), ref)
    too_many = W.make_uniform(B.STATIC_MAX_P + 1, 1)
    with pytest.raises(B.TunaError, match="RANGE"):
        B.direct_alltoallv_static(too_many.P, 1, too_many.sendcounts, send, want)
    # (sizes over the stated limits are refused before the buffers are looked at:
    # that case needs no GPU and no buffers, and is covered with the host-side checks)
    with pytest.raises(B.TunaError, match="OVERLAP"):
        B.direct_alltoallv_static(wl.P, 1, wl.sendcounts, send, send)


def test_a_stream_under_capture_is_refused():
    """The call uploads host arrays with asynchronous copies; recorded into a graph they
    would be read again at every replay.  It must refuse, record nothing, and leave the
    capture usable."""
    wl = W.make_random(9, 200, elem_size=1, seed=44)
    send, want = plan_based(wl)
    recv = wl.make_recv("cuda", fill=CANARY)
    B.direct_alltoallv_static(wl.P, wl.elem_size, wl.sendcounts, send, recv)   # the set-up call, eager
    torch.cuda.synchronize()
    st = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    filler = torch.zeros(8, device="cuda")
    with torch.cuda.stream(st):
        graph.capture_begin()
        try:
            with pytest.raises(B.TunaError, match="INVALID_ARG"):
                B.direct_alltoallv_static(wl.P, wl.elem_size, wl.sendcounts, send, recv, stream=st)
            filler.add_(1)
        finally:
            graph.capture_end()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(recv, want) and float(filler.sum()) == 8.0

"""The allocation-free direct exchange against the plan-based one.

Some users of this library run where device allocation is off limits: the
framework around them has handed all GPU memory to its own pool, or their
serving loop forbids cudaMalloc after start-up because it stalls every stream.
They call ``tuna_direct_alltoallv_static``, which keeps its tables in a fixed
array inside the library.  This file checks, through the C ABI, that it writes
exactly the bytes ``tuna_direct_alltoallv`` writes, on two calls in a row (the
second one finds the first one's tables in the shared array).  It is collected
last, so that a run stopping at the first failure has run everything else.
"""
import numpy as np
import pytest
import torch

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


def test_large_blocks_and_limits():
    wl = W.make_random(4, 3_000_000, elem_size=1, seed=43)
    send, want = plan_based(wl)
    assert torch.equal(no_alloc(wl, send), want)
    too_many = W.make_uniform(B.STATIC_MAX_P + 1, 1)
    with pytest.raises(B.TunaError, match="RANGE"):
        B.direct_alltoallv_static(too_many.P, 1, too_many.sendcounts, send, want)
    # 5 GiB of blocks: over the stated limit, rejected before anything is launched
    huge = np.zeros((2, 2), dtype=np.int64)
    huge[0, 1] = 5 << 30
    with pytest.raises(B.TunaError, match="RANGE"):
        B.direct_alltoallv_static(2, 1, huge, 1 << 20, (1 << 20) + (6 << 30))
    with pytest.raises(B.TunaError, match="OVERLAP"):
        B.direct_alltoallv_static(wl.P, 1, wl.sendcounts, send, send)

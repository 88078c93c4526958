"""The sharded exchange (one group of ranks per GPU) against the CPU oracle, on ONE GPU.

Every GPU of the real thing is stood in for by its own buffers, its own plan and its
own stream on the same device; the "other GPUs' receive buffers" are simply the other
shards' buffers.  No kernel of the sharded path waits for another one, so the shards
may run in any order or at the same time.  What cannot be seen here is the link between
GPUs and the mapping of memory between processes on different devices; a two-process run
on the one device covers the handles and the orchestration."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from paper_2411_02581_b200 import binding as B
from paper_2411_02581_b200 import workloads as W

pytestmark = pytest.mark.gpu

CANARY = 0xA5
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def shard_buffers(wl, G):
    """The global buffers of a workload cut into one piece per GPU (at the first region of
    each group), and every rank's region base inside its GPU's piece."""
    l, E = wl.P // G, wl.elem_size
    first = np.arange(G) * l
    cut_s = [int(wl.sendbase[p]) * E for p in first] + [wl.send_bytes]
    cut_r = [int(wl.recvbase[p]) * E for p in first] + [wl.recv_bytes]
    grp = np.arange(wl.P) // l
    sb = wl.sendbase - wl.sendbase[first][grp]
    rb = wl.recvbase - wl.recvbase[first][grp]
    return cut_s, cut_r, sb, rb


def run_sharded(wl, G, radix, explicit_bases=True, phases=B.SHARD_LOCAL | B.SHARD_GLOBAL, two_calls=False):
    cut_s, cut_r, sb, rb = shard_buffers(wl, G)
    send = wl.make_send("cuda")
    sends = [send[cut_s[n]:cut_s[n + 1]].clone() for n in range(G)]
    recvs = [torch.full((max(cut_r[n + 1] - cut_r[n], 16),), CANARY, dtype=torch.uint8, device="cuda")
             for n in range(G)]
    kw = dict(sendbase=sb, recvbase=rb) if explicit_bases else {}
    plans = [B.Plan(wl.P, radix, elem_size=wl.elem_size, sendcounts=wl.sendcounts, sdispls=wl.sdispls,
                    rdispls=wl.rdispls, shard=(G, n), **kw) for n in range(G)]
    streams = [torch.cuda.Stream() for _ in range(G)]
    torch.cuda.synchronize()
    for n, plan in enumerate(plans):
        assert plan.shard_extents(n) == plan.extents()[:2]
        for m in range(G):
            se, re = plan.shard_extents(m)
            assert se <= cut_s[m + 1] - cut_s[m] and re <= cut_r[m + 1] - cut_r[m]
        plan.alloc_workspace()
        if two_calls:   # local part everywhere first, then the pushes: the two halves of an exchange
            plan.shard_alltoallv(sends[n], recvs, phases=B.SHARD_LOCAL, stream=streams[n])
        else:
            plan.shard_alltoallv(sends[n], recvs, phases=phases, stream=streams[n])
    if two_calls:
        for n, plan in enumerate(plans):
            plan.shard_alltoallv(sends[n], recvs, phases=B.SHARD_GLOBAL, stream=streams[n])
    torch.cuda.synchronize()
    got = torch.cat([recvs[n][:cut_r[n + 1] - cut_r[n]] for n in range(G)]).cpu().numpy()
    return got, plans


def oracle_hier(wl, l, G, rl):
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    return oracle.tuna_hier(wl, l, G, rl, max(2, G), send, recv, want_after_local=True)


SHARDED = [(P, G, r) for P, G in [(8, 2), (8, 4), (12, 3), (16, 2), (16, 4), (20, 4), (6, 6), (5, 1), (64, 4), (64, 8)]
           for r in sorted({0, 2, max(2, P // G)})]


@pytest.mark.parametrize("P,G,radix", SHARDED)
def test_sharded_exchange_matches_the_oracle(P, G, radix):
    """g = 2, 3, 4, ... GPUs' worth of shards on one device: assembled receive buffers against
    the hierarchical oracle with one group per GPU and the coalesced inter-group exchange;
    every shard's round table against the oracle run on that shard's rows alone."""
    l = P // G
    wl = W.make_random(P, 400, elem_size=2, seed=13 * P + G + radix, zero_frac=0.25, gaps=True)
    rl = radix if radix else max(2, l)
    ref, rounds, _, after = oracle_hier(wl, l, G, rl)
    got, plans = run_sharded(wl, G, radix)
    assert np.array_equal(got, ref)
    total = np.zeros(len(rounds), dtype=np.int64)
    for n, plan in enumerate(plans):
        mine = plan.rounds()
        assert len(mine) == len(rounds)
        # what this GPU sends: the oracle on a count matrix that keeps only its rows
        only = wl.sendcounts.copy()
        only[:n * l] = 0
        only[(n + 1) * l:] = 0
        wn = W._finish("shard", P, wl.elem_size, 1, only)
        _, rn, _, _ = oracle_hier(wn, l, G, rl)
        table = B.shard_round_table(P, G, n, radix, wl.elem_size, wl.sendcounts)
        for k, (a, row, rown) in enumerate(zip(mine, rounds, rn)):
            assert (a["level"], a["x"], a["z"]) == tuple(int(v) for v in row[:3])
            assert a["bytes"] == rown[oracle.RS_BYTES_SENT]
            assert (table[k]["level"], table[k]["x"], table[k]["z"], table[k]["bytes"]) == \
                (a["level"], a["x"], a["z"], a["bytes"])
            total[k] += a["bytes"]
    assert np.array_equal(total, rounds[:, oracle.RS_BYTES_SENT])


@pytest.mark.parametrize("P,G,radix", [(15, 3, 2), (16, 4, 2), (64, 8, 8)])
def test_local_part_alone_leaves_the_own_groups_blocks(P, G, radix):
    """After the local phases the receive buffers hold exactly the blocks from ranks of the
    own group (the state the paper's Fig. 5 describes); the pushes then complete them."""
    l = P // G
    wl = W.make_random(P, 300, elem_size=1, seed=P + G, zero_frac=0.2, gaps=True)
    ref, _, _, after = oracle_hier(wl, l, G, radix)
    got, _ = run_sharded(wl, G, radix, phases=B.SHARD_LOCAL)
    assert np.array_equal(got, after)
    got, _ = run_sharded(wl, G, radix, two_calls=True)
    assert np.array_equal(got, ref)


def test_packed_bases_and_recount():
    """NULL bases = every GPU's regions packed from offset 0 of its own buffers; an update
    with new counts re-plans the shard."""
    P, G = 24, 4
    wl = W.make_random(P, 500, elem_size=4, seed=3, zero_frac=0.3)          # packed: regions back to back
    ref, _, _, _ = oracle_hier(wl, P // G, G, 2)
    got, plans = run_sharded(wl, G, 2, explicit_bases=False)
    assert np.array_equal(got, ref)
    sb, rb, se, re = B.shard_layout(P, G, wl.elem_size, wl.sendcounts)
    cut_s, cut_r, esb, erb = shard_buffers(wl, G)
    assert np.array_equal(sb, esb) and np.array_equal(rb, erb)
    assert [int(v) for v in se] == [cut_s[n + 1] - cut_s[n] for n in range(G)]
    assert [int(v) for v in re] == [cut_r[n + 1] - cut_r[n] for n in range(G)]
    wl2 = W.make_random(P, 300, elem_size=4, seed=4, zero_frac=0.1)
    ref2, _, _, _ = oracle_hier(wl2, P // G, G, 2)
    cut_s, cut_r, _, _ = shard_buffers(wl2, G)
    send = wl2.make_send("cuda")
    recvs = [torch.full((max(cut_r[n + 1] - cut_r[n], 16),), CANARY, dtype=torch.uint8, device="cuda")
             for n in range(G)]
    for n, plan in enumerate(plans):
        plan.update_counts(wl2.sendcounts)
        plan.alloc_workspace()
        plan.shard_alltoallv(send[cut_s[n]:cut_s[n + 1]].clone(), recvs)
    torch.cuda.synchronize()
    got2 = torch.cat([recvs[n][:cut_r[n + 1] - cut_r[n]] for n in range(G)]).cpu().numpy()
    assert np.array_equal(got2, ref2)


def test_sharded_plan_argument_checks():
    wl = W.make_random(8, 50, seed=9)
    with pytest.raises(B.TunaError, match="BAD_HIERARCHY"):
        B.Plan(8, 2, sendcounts=wl.sendcounts, shard=(3, 0))
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        B.Plan(8, 2, sendcounts=wl.sendcounts, shard=(2, 2))
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        B.Plan(8, 2, sendcounts=wl.sendcounts, shard=(2, 0), flags=B.FLAG_CLASSIC_ROTATE)
    plan = B.Plan(8, 2, sendcounts=wl.sendcounts, shard=(2, 0))
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        plan.alltoallv(buf, buf)                       # a sharded plan only runs through its own call
    with pytest.raises(B.TunaError, match="WORKSPACE"):
        plan.shard_alltoallv(buf[:4096], [buf[8192:], buf[32768:]])
    plan.alloc_workspace()
    with pytest.raises(B.TunaError, match="OVERLAP"):
        plan.shard_alltoallv(buf, [buf, buf[32768:]])
    d_counts = torch.from_numpy(wl.sendcounts).cuda()
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        plan.update_counts_device(d_counts)


def test_two_processes_share_one_gpu():
    """The orchestration as it runs under a launcher, with two processes on the one device:
    counts all-gathered, receive buffers exported and mapped through memory handles, the
    push into the other process's buffer, host-level barriers (the NCCL backend needs one
    GPU per process, so this run uses gloo)."""
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29631", PYTHONPATH=ROOT)
    procs = [subprocess.Popen([sys.executable, os.path.join(ROOT, "tests", "sharded_worker.py"), str(r), "2"],
                              env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
             for r in range(2)]
    outs = []
    for p in procs:
        try:
            out, _ = p.communicate(timeout=300)
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
        outs.append(out)
    for r, p in enumerate(procs):
        assert p.returncode == 0, outs[r]
        assert "sharded ok" in outs[r], outs[r]

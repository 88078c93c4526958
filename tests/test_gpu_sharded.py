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


def oracle_brute(wl):
    return oracle.bruteforce(wl, wl.make_send().numpy(), wl.make_recv(fill=CANARY).numpy().copy())


def test_large_blocks_cross_between_shards(monkeypatch):
    """Megabyte blocks: the pushes run the large-block build of the mover (chunks inside one
    block, plain and skewed) with destinations in the other shards' buffers."""
    monkeypatch.setenv("TUNA_SMALL_LIST_BYTES", "0")      # (lists this short would otherwise take the other build)
    wl = W.make_random(8, 2_100_000, elem_size=1, seed=5, zero_frac=0.1, gaps=True)      # odd byte counts: skewed
    assert wl.payload_bytes_total > 48 << 20
    ref = oracle_brute(wl)
    for G in (2, 4):
        got, plans = run_sharded(wl, G, 2)
        assert np.array_equal(got, ref)
        assert any(p.last_launches() > p.last_small_launches() for p in plans)            # the large build did run
    aligned = W.make_c4(P=16, tokens=256, hidden=2048)                                  # 4 KiB rows, aligned
    got, _ = run_sharded(aligned, 4, 0)
    assert np.array_equal(got, oracle_brute(aligned))


@pytest.mark.parametrize("elem", [1, 3, 8, 48])
def test_element_sizes(elem):
    wl = W.make_random(12, 300, elem_size=elem, seed=elem, zero_frac=0.2, gaps=True)
    ref = oracle_brute(wl)
    for G, r in ((3, 2), (6, 0), (12, 2)):
        got, _ = run_sharded(wl, G, r)
        assert np.array_equal(got, ref)


def test_c5_over_eight_shards():
    """The 2048-rank workload of tiny unaligned blocks, 256 ranks per shard: every byte
    against the definition of the exchange, the shards' rounds against the oracle's."""
    wl = W.make_c5()
    l, G = wl.P // 8, 8
    ref, rounds, _, _ = oracle_hier(wl, l, G, l)
    got, plans = run_sharded(wl, G, 0, explicit_bases=False)
    assert np.array_equal(got, ref)
    total = np.zeros(len(rounds), dtype=np.int64)
    for plan in plans:
        total += np.array([r["bytes"] for r in plan.rounds()])
    assert np.array_equal(total, rounds[:, oracle.RS_BYTES_SENT])
    # every shard's launches: one local phase (with the self blocks) and the push
    assert all(p.last_launches() == 2 for p in plans)


def test_timing_kinds_and_self_blocks_only():
    wl = W.make_random(8, 200, elem_size=2, seed=21)
    plans = None
    got, plans = run_sharded(wl, 8, 2)                       # one rank per shard: no local phase at all
    assert np.array_equal(got, oracle_brute(wl))
    diag = W._finish("diag", 8, 2, 1, np.diag(np.arange(1, 9)).astype(np.int64))    # nothing but self blocks
    got, plans = run_sharded(diag, 4, 2)
    assert np.array_equal(got, oracle_brute(diag))
    wl2 = W.make_random(16, 200, elem_size=2, seed=22)
    cut_s, cut_r, sb, rb = shard_buffers(wl2, 2)
    plan = B.Plan(16, 4, elem_size=2, sendcounts=wl2.sendcounts, sdispls=wl2.sdispls, rdispls=wl2.rdispls,
                  sendbase=sb, recvbase=rb, shard=(2, 0))
    plan.alloc_workspace()
    plan.enable_timing(True)
    send = wl2.make_send("cuda")[cut_s[0]:cut_s[1]].clone()
    recvs = [torch.zeros(max(cut_r[n + 1] - cut_r[n], 16), dtype=torch.uint8, device="cuda") for n in range(2)]
    plan.shard_alltoallv(send, recvs)
    t = plan.get_timing()
    assert t["round_local"]["launches"] == 2 and t["round_global"]["launches"] == 1     # radix 4 over 8 ranks: 2 local phases
    mine = plan.rounds()
    assert t["round_global"]["bytes"] == sum(r["bytes"] for r in mine if r["level"] == 1)


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
    # and from a count matrix in device memory: bases and buffer sizes worked out on the device
    wl3 = W.make_random(P, 700, elem_size=4, seed=6, zero_frac=0.4)
    ref3, rounds3, _, _ = oracle_hier(wl3, P // G, G, 2)
    cut_s, cut_r, _, _ = shard_buffers(wl3, G)
    d_counts = torch.from_numpy(wl3.sendcounts).cuda()
    send = wl3.make_send("cuda")
    recvs = [torch.full((max(cut_r[n + 1] - cut_r[n], 16),), CANARY, dtype=torch.uint8, device="cuda")
             for n in range(G)]
    total = np.zeros(len(rounds3), dtype=np.int64)
    for n, plan in enumerate(plans):
        plan.update_counts_device(d_counts)
        for m in range(G):
            assert plan.shard_extents(m) == (cut_s[m + 1] - cut_s[m], cut_r[m + 1] - cut_r[m])
        assert plan.extents() == (cut_s[n + 1] - cut_s[n], cut_r[n + 1] - cut_r[n], wl3.payload_bytes_total)
        plan.alloc_workspace()
        plan.shard_alltoallv(send[cut_s[n]:cut_s[n + 1]].clone(), recvs)
        total += np.array([r["bytes"] for r in plan.rounds()])
    torch.cuda.synchronize()
    got3 = torch.cat([recvs[n][:cut_r[n + 1] - cut_r[n]] for n in range(G)]).cpu().numpy()
    assert np.array_equal(got3, ref3)
    assert np.array_equal(total, rounds3[:, oracle.RS_BYTES_SENT])
    neg = d_counts.clone()
    neg[3, 5] = -2
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        plans[0].update_counts_device(neg)
    plans[0].update_counts_device(d_counts)                  # and the plan recovers


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


def test_two_processes_share_one_gpu():
    """The orchestration as it runs under a launcher, with two processes on the one device:
    counts all-gathered, receive buffers exported and mapped through memory handles, the
    push into the other process's buffer, host-level barriers (the NCCL backend needs one
    GPU per process, so this run uses gloo)."""
    import socket
    with socket.socket() as sock:                      # a port that is free right now
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), PYTHONPATH=ROOT)
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

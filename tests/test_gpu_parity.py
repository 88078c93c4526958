"""CUDA path vs CPU oracle, bit-exact, through the C ABI.  Needs a GPU."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2411_02581_b200 import binding as B
from paper_2411_02581_b200 import workloads as W

pytestmark = pytest.mark.gpu

CANARY = 0xA5


def oracle_flat(wl, r, want_sizes=False):
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    return oracle.tuna_flat(wl, r, send, recv, want_sizes=want_sizes)


def oracle_hier(wl, Q, N, rl, rg):
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    return oracle.tuna_hier(wl, Q, N, rl, rg, send, recv)


def oracle_brute(wl):
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    return oracle.bruteforce(wl, send, recv)


def gpu_run(wl, radix, l=None, g=1, rg=2, flags=0, direct=False, explicit=True, pass_args=True,
            misalign=0, block_count=0):
    """Run the exchange on the GPU; returns (recv bytes as numpy, plan).
    ``misalign`` shifts both device buffers by that many bytes off 256-byte alignment."""
    send0 = wl.make_send("cuda")
    recv0 = wl.make_recv("cuda", fill=CANARY)
    if misalign:
        sbuf = torch.empty(send0.numel() + 64, dtype=torch.uint8, device="cuda")
        rbuf = torch.full((recv0.numel() + 64,), CANARY, dtype=torch.uint8, device="cuda")
        send = sbuf[misalign:misalign + send0.numel()]
        send.copy_(send0)
        recv = rbuf[misalign:misalign + recv0.numel()]
    else:
        send, recv = send0, recv0
    plan = B.plan_for(wl, radix, l=l, g=g, radix_global=rg, flags=flags, explicit_layout=explicit,
                      block_count=block_count)
    plan.alloc_workspace()
    args = {}
    if pass_args and explicit:
        args = dict(sendcounts=wl.sendcounts, sdispls=wl.sdispls, recvcounts=wl.recvcounts,
                    rdispls=wl.rdispls)
    if direct:
        plan.direct_alltoallv(send, recv, **args)
    else:
        plan.alltoallv(send, recv, **args)
    torch.cuda.synchronize()
    if misalign:
        assert bool((rbuf[:misalign] == CANARY).all()) and bool((rbuf[misalign + recv0.numel():] == CANARY).all())
    return recv.cpu().numpy(), plan


def check_rounds(plan, rounds):
    got = plan.rounds()
    assert len(got) == len(rounds)
    for g, row in zip(got, rounds):
        assert (g["level"], g["x"], g["z"]) == tuple(int(v) for v in row[:3])
        assert g["units"] == row[oracle.RS_UNITS]
        assert g["bytes"] == row[oracle.RS_BYTES_SENT] == row[oracle.RS_BYTES_RECV]


FLAT = [(P, r) for P in (1, 2, 3, 5, 8, 9, 16, 17) for r in sorted({2, 3, max(2, P // 2), max(2, P)})
        if r <= max(2, P)]
FLAT += [(33, 2), (33, 6), (64, 4), (100, 10), (130, 2), (130, 130)]


@pytest.mark.parametrize("P,r", FLAT)
@pytest.mark.parametrize("flags", [B.FLAG_DIRECT_TO_R, B.FLAG_CLASSIC_ROTATE])
def test_flat_small(P, r, flags):
    """Unaligned byte counts, gaps with canaries, every radix class, both placements."""
    wl = W.make_random(P, 300, elem_size=1, seed=1000 + P, zero_frac=0.25, gaps=True)
    ref, rounds, _, _ = oracle_flat(wl, r)
    got, plan = gpu_run(wl, r, flags=flags)
    assert np.array_equal(got, ref)
    check_rounds(plan, rounds)
    got_d, _ = gpu_run(wl, r, direct=True)
    assert np.array_equal(got_d, ref)


@pytest.mark.parametrize("elem", [1, 2, 3, 4, 8, 16, 48])
@pytest.mark.parametrize("misalign", [0, 1, 4, 7])
def test_element_sizes_and_buffer_alignment(elem, misalign):
    wl = W.make_random(12, 700, elem_size=elem, seed=elem, zero_frac=0.1, gaps=True)
    ref = oracle_brute(wl)
    for r in (2, 4, 12):
        got, _ = gpu_run(wl, r, misalign=misalign)
        assert np.array_equal(got, ref)
    got, _ = gpu_run(wl, 3, flags=B.FLAG_CLASSIC_ROTATE, misalign=misalign)
    assert np.array_equal(got, ref)
    got, _ = gpu_run(wl, 2, direct=True, misalign=misalign)
    assert np.array_equal(got, ref)


def test_large_blocks_span_many_chunks():
    """Blocks far larger than one CTA's chunk, plus a ragged tail."""
    wl = W.make_random(6, 3_000_000, elem_size=1, seed=77, zero_frac=0.2)
    ref, rounds, _, _ = oracle_flat(wl, 2)
    for flags in (0, B.FLAG_CLASSIC_ROTATE):
        got, plan = gpu_run(wl, 2, flags=flags)
        assert np.array_equal(got, ref)
    check_rounds(plan, rounds)
    got, _ = gpu_run(wl, 6, direct=True)
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("misalign", [0, 5])
def test_large_skewed_blocks(misalign):
    """Megabyte blocks of odd byte counts in lists large enough for the large-block
    build: chunks inside one block whose source is skewed against its destination
    (one aligned load per vector, the neighbour's words by shuffle)."""
    wl = W.make_random(12, 2_100_000, elem_size=1, seed=91, zero_frac=0.1, gaps=True)
    assert wl.payload_bytes_total > 96 << 20
    ref, rounds, _, _ = oracle_flat(wl, 3)
    for flags in (0, B.FLAG_CLASSIC_ROTATE):
        got, plan = gpu_run(wl, 3, flags=flags, misalign=misalign)
        assert np.array_equal(got, ref)
    check_rounds(plan, rounds)
    got, _ = gpu_run(wl, 12, misalign=misalign)
    assert np.array_equal(got, ref)
    got, _ = gpu_run(wl, 2, direct=True, misalign=misalign)
    assert np.array_equal(got, ref)
    wl8 = W.make_random(12, 260_000, elem_size=8, seed=92)            # skew of 0 or 8 bytes only
    got, _ = gpu_run(wl8, 12, misalign=misalign)
    assert np.array_equal(got, oracle_brute(wl8))


@pytest.mark.parametrize("kw", [dict(radix=2), dict(radix=8), dict(radix=600), dict(radix=2, flags=B.FLAG_CLASSIC_ROTATE),
                                dict(radix=5, l=20, g=30, rg=6), dict(radix=600, direct=True)])
def test_ranks_that_send_or_receive_nothing(kw):
    """Runs of tens of thousands of empty blocks inside a chunk's descriptors (the mover
    finds their end by doubling steps and bisection, not batch by batch)."""
    wl = W.make_silent_ranks(600, 90, 150, 520, 80, 410, gaps=True)
    assert (wl.sendcounts == 0).mean() > 0.8
    kw = dict(kw)
    got, _ = gpu_run(wl, kw.pop("radix"), **kw)
    assert np.array_equal(got, oracle_brute(wl))


def test_bulk_copy_route():
    """TUNA_FLAG_BULK_COPY: chunks inside large aligned blocks go through
    cp.async.bulk; same bytes, and no kernel gives up a wait."""
    aligned = W.make_c4(P=16, tokens=256, hidden=512)          # 1 KiB rows, blocks of ~32 KiB
    ragged = W.make_random(6, 3_000_000, elem_size=1, seed=78, zero_frac=0.2)   # unaligned: falls back
    for wl in (aligned, ragged):
        ref = oracle_brute(wl)
        for r, flags in ((2, B.FLAG_BULK_COPY), (4, B.FLAG_BULK_COPY | B.FLAG_CLASSIC_ROTATE),
                         (wl.P, B.FLAG_BULK_COPY)):
            got, plan = gpu_run(wl, r, flags=flags)
            assert np.array_equal(got, ref)
            assert plan.device_status() == 0
        got, plan = gpu_run(wl, 2, flags=B.FLAG_BULK_COPY, direct=True)
        assert np.array_equal(got, ref) and plan.device_status() == 0


HIER = [(Q, N, rl, rg) for Q, N in [(1, 4), (4, 1), (2, 2), (3, 4), (5, 3), (4, 4), (8, 4), (6, 5)]
        for rl in sorted({2, max(2, Q)}) for rg in sorted({2, 3, max(2, N)})
        if rl <= max(2, Q) and rg <= max(2, N)]


@pytest.mark.parametrize("Q,N,rl,rg", HIER)
def test_hier_small(Q, N, rl, rg):
    P = Q * N
    wl = W.make_random(P, 200, elem_size=2, seed=31 * P + rl + rg, zero_frac=0.2, gaps=True)
    ref, rounds, _, _ = oracle_hier(wl, Q, N, rl, rg)
    for flags in (0, B.FLAG_CLASSIC_ROTATE):
        got, plan = gpu_run(wl, rl, l=Q, g=N, rg=rg, flags=flags)
        assert np.array_equal(got, ref)
        check_rounds(plan, rounds)


@pytest.mark.parametrize("P,r", [(8, 2), (9, 3), (16, 4), (20, 5), (64, 8), (5, 5), (33, 33), (70, 70), (64, 64)])
def test_metadata_and_prefix_sums(P, r):
    """Descriptor tables of every digit phase: sizes equal the oracle's
    message-passed metadata, positions equal its running sums."""
    wl = W.make_random(P, 500, elem_size=3, seed=P + r, zero_frac=0.3)
    _, _, _, _, sizes = oracle_flat(wl, r, want_sizes=True)
    plan = B.plan_for(wl, r)
    assert plan.num_phases() == sizes.shape[0]
    work_off = 0
    for x in range(plan.num_phases()):
        moving = [o for o in range(P) if (o // r ** x) % r != 0]
        arrived = [o for o in moving if o < r ** (x + 1)]      # no non-zero digit above x
        onward = [o for o in moving if o >= r ** (x + 1)]
        assert moving == arrived + onward                      # the arrived ones come first
        # blocks that travel on: this phase's region of the workspace
        t = plan.phase_tables(x, B.PART_KEEP)
        exp_len = sizes[x][:, onward]                          # receive-side order (rank, offset)
        assert np.array_equal(t["len"].reshape(P, len(onward)), exp_len)
        scan, tot = oracle.segmented_exclusive_scan(exp_len, 16)
        base, _ = oracle.segmented_exclusive_scan(tot.reshape(1, P), 1)
        exp_pos = scan + base.reshape(P, 1)
        assert np.array_equal(t["pos"].reshape(P, len(onward)), exp_pos)
        info = plan.phase_info(x, B.PART_KEEP)
        assert info["bytes"] == exp_len.sum() and info["stream_bytes"] == tot.sum()
        assert np.array_equal(t["dst"].reshape(P, len(onward)), (2 << 56) | (work_off + exp_pos))
        work_off += (int(tot.sum()) + 255) // 256 * 256
        # blocks that have arrived: straight into the receive buffer
        t = plan.phase_tables(x, B.PART_DELIVER)
        exp_len = sizes[x][:, arrived]
        assert np.array_equal(t["len"].reshape(P, len(arrived)), exp_len)
        spaced = (exp_len + 15) // 16 * 16 + 16 * (exp_len > 0)
        scan, tot = oracle.segmented_exclusive_scan(spaced, 1)
        base, _ = oracle.segmented_exclusive_scan(tot.reshape(1, P), 1)
        assert np.array_equal(t["pos"].reshape(P, len(arrived)), scan + base.reshape(P, 1))
        assert plan.phase_info(x, B.PART_DELIVER)["bytes"] == exp_len.sum()
        dst = t["dst"].reshape(P, len(arrived))
        for p in range(P):
            for j, o in enumerate(arrived):
                s = (p - o) % P
                assert dst[p, j] == (1 << 56) | int(wl.recvbase[p] + wl.rdispls[p, s]) * wl.elem_size
    assert plan.workspace_bytes() == work_off
    # one phase that delivers everything: it doubles as the direct exchange's list
    assert plan.phase_info(-2)["entries"] == (0 if r >= P else P * P)
    # classic mode keeps every block in the workspace and rotates at the end
    classic = B.plan_for(wl, r, flags=B.FLAG_CLASSIC_ROTATE)
    for x in range(classic.num_phases()):
        moving = [o for o in range(P) if (o // r ** x) % r != 0]
        t = classic.phase_tables(x, B.PART_KEEP)
        assert np.array_equal(t["len"].reshape(P, len(moving)), sizes[x][:, moving])
        assert classic.phase_info(x, B.PART_DELIVER)["entries"] == 0
    rot = classic.phase_tables(-1)
    assert np.array_equal(rot["len"].reshape(P, P), sizes[-1])   # every block, in slot order

def _digit(v, r, x):
    return (v // r ** x) % r


@pytest.mark.parametrize("Q,N,rl,rg", [(5, 3, 2, 3), (4, 4, 2, 2), (3, 4, 3, 2), (6, 5, 2, 3), (8, 4, 8, 4),
                                       (16, 16, 4, 4), (32, 8, 32, 8)])
def test_hier_metadata_and_prefix_sums(Q, N, rl, rg):
    """Descriptor tables of every local and global digit phase of a hierarchical plan:
    sizes equal the oracle's message-passed metadata (the global phases' against the
    sub-block sizes of its compacted super-blocks), positions equal its running sums,
    and every block is read from where the previous phase put it."""
    P = Q * N
    wl = W.make_random(P, 300, elem_size=3, seed=17 * P + rl + rg, zero_frac=0.3, gaps=True)
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    _, _, sz_local, usz_compact, usz_global = oracle.tuna_hier_tables(wl, Q, N, rl, rg, send, recv)
    plan = B.plan_for(wl, rl, l=Q, g=N, radix_global=rg)
    wloc, wglo = sz_local.shape[0], usz_global.shape[0]
    assert plan.num_phases() == wloc + wglo
    E = wl.elem_size
    ranks = np.arange(P)
    n_of, q_of = ranks // Q, ranks % Q

    def recv_loc(p, origin):
        return (1 << 56) | int(wl.recvbase[p] + wl.rdispls[p, origin]) * E

    # where every rank keeps the block of slot (io, jo): at first in its send region
    loc = {}
    for p in range(P):
        for io in range(N):
            for jo in range(Q):
                dest = ((n_of[p] + io) % N) * Q + (q_of[p] + jo) % Q
                loc[p, io, jo] = int(wl.sendbase[p] + wl.sdispls[p, dest]) * E
    work_off = 0
    for f in range(wloc + wglo):
        level, x = (0, f) if f < wloc else (1, f - wloc)
        if level == 0:
            moving = [jo for jo in range(Q) if _digit(jo, rl, x) != 0]
            row = [(io, jo) for io in range(N) for jo in moving]
            arrived = [(0, jo) for jo in moving if jo < rl ** (x + 1)]       # own group, no digit above x
            # the oracle's table is by destination group; a slot names the group offset
            size = lambda p, io, jo: sz_local[x, p, (n_of[p] + io) % N, jo]
            sender = lambda p, io, jo: n_of[p] * Q + (q_of[p] - _digit(jo, rl, x) * rl ** x) % Q
        else:
            moving = [io for io in range(N) if _digit(io, rg, x) != 0]
            row = [(io, jo) for io in moving for jo in range(Q)]
            arrived = [(io, jo) for io in moving if io < rg ** (x + 1) for jo in range(Q)]
            # a super-block's parts are listed by source local id q' = q - jo
            size = lambda p, io, jo: usz_global[x, p, io, (q_of[p] - jo) % Q]
            sender = lambda p, io, jo: ((n_of[p] - _digit(io, rg, x) * rg ** x) % N) * Q + q_of[p]
        assert row[:len(arrived)] == arrived                                # the arrived ones come first
        onward = row[len(arrived):]
        new_loc = {}
        for part, slots in ((B.PART_KEEP, onward), (B.PART_DELIVER, arrived)):
            t = plan.phase_tables(f, part)
            m = len(slots)
            exp_len = np.array([[size(p, io, jo) for io, jo in slots] for p in range(P)], dtype=np.int64).reshape(P, m)
            assert np.array_equal(t["len"].reshape(P, m), exp_len)
            if level == 1 and x == 0:
                # what the first global phase gathers is what the compaction laid out at the sender
                comp = np.array([[usz_compact[sender(p, io, jo), io, (q_of[p] - jo) % Q] for io, jo in slots]
                                 for p in range(P)], dtype=np.int64).reshape(P, m)
                assert np.array_equal(exp_len, comp)
            spaced = (exp_len + 15) // 16 * 16 + (16 * (exp_len > 0) if part == B.PART_DELIVER else 0)
            scan, tot = oracle.segmented_exclusive_scan(spaced, 1)
            base, _ = oracle.segmented_exclusive_scan(tot.reshape(1, P), 1)
            exp_pos = scan + base.reshape(P, 1)
            assert np.array_equal(t["pos"].reshape(P, m), exp_pos)
            info = plan.phase_info(f, part)
            assert info["bytes"] == exp_len.sum() and info["level"] == level and info["x"] == x
            src, dst = t["src"].reshape(P, m), t["dst"].reshape(P, m)
            for p in range(P):
                for j, (io, jo) in enumerate(slots):
                    assert src[p, j] == loc[sender(p, io, jo), io, jo]
                    if part == B.PART_KEEP:
                        assert dst[p, j] == (2 << 56) | (work_off + int(exp_pos[p, j]))
                    else:
                        origin = ((n_of[p] - io) % N) * Q + (q_of[p] - jo) % Q
                        assert dst[p, j] == recv_loc(p, origin)
                    new_loc[p, io, jo] = int(dst[p, j])
            if part == B.PART_KEEP:
                assert info["stream_bytes"] == tot.sum()
                work_off += (int(tot.sum()) + 255) // 256 * 256
        loc.update(new_loc)
    assert plan.workspace_bytes() == work_off
    # at the end every block but the self blocks sits at its place in the receive buffer
    for p in range(P):
        for io in range(N):
            for jo in range(Q):
                if io or jo:
                    assert loc[p, io, jo] == recv_loc(p, ((n_of[p] - io) % N) * Q + (q_of[p] - jo) % Q)


def test_radix_zero_chooses_one_hop_per_level():
    wl = W.make_random(12, 100, elem_size=2, seed=5, zero_frac=0.2, gaps=True)
    ref = oracle_brute(wl)
    got, plan = gpu_run(wl, 0)
    assert np.array_equal(got, ref) and plan.num_phases() == 1 and plan.num_rounds() == 11
    got, plan = gpu_run(wl, 0, l=4, g=3, rg=0)
    assert np.array_equal(got, ref) and plan.num_phases() == 2 and plan.num_rounds() == 3 + 2


def test_packed_layout_defaults_match_explicit():
    """NULL displacement arrays mean 'packed'; the device-side scans must give
    the same layout the generator computed on the host."""
    wl = W.make_random(19, 90, elem_size=4, seed=8, zero_frac=0.2)
    ref = oracle_brute(wl)
    got, plan = gpu_run(wl, 3, explicit=False)
    assert np.array_equal(got, ref)
    assert plan.extents() == (wl.send_bytes, wl.recv_bytes, wl.payload_bytes_total)
    d = plan.phase_tables(-2)
    assert np.array_equal(d["len"].reshape(19, 19), wl.sendcounts.T * 4)
    exp_dst = (wl.recvbase[:, None] + wl.rdispls) * 4 + (1 << 56)
    assert np.array_equal(d["dst"].reshape(19, 19), exp_dst)


def test_call_time_validation():
    wl = W.make_random(6, 50, seed=4)
    send = wl.make_send("cuda")
    recv = wl.make_recv("cuda")
    plan = B.plan_for(wl, 2)
    with pytest.raises(B.TunaError, match="WORKSPACE"):
        plan.alltoallv(send, recv)
    plan.alloc_workspace()
    bad = wl.sendcounts.copy()
    bad[0, 1] += 1
    with pytest.raises(B.TunaError, match="COUNT_MISMATCH"):
        plan.alltoallv(send, recv, sendcounts=bad)
    with pytest.raises(B.TunaError, match="COUNT_MISMATCH"):
        plan.alltoallv(send, recv, recvcounts=wl.sendcounts + np.eye(6, dtype=np.int64))
    with pytest.raises(B.TunaError, match="COUNT_MISMATCH"):
        plan.alltoallv(send, recv, rdispls=wl.rdispls + 1)
    both = torch.zeros(wl.send_bytes + wl.recv_bytes, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.TunaError, match="OVERLAP"):
        plan.alltoallv(both, both[8:])
    before = recv.clone()
    torch.cuda.synchronize()
    assert torch.equal(recv, before)            # failed calls wrote nothing
    plan.alltoallv(send, recv, wl.sendcounts, wl.sdispls, wl.recvcounts, wl.rdispls)
    torch.cuda.synchronize()
    assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl))


def test_update_counts_and_rerun():
    wl1 = W.make_random(10, 400, seed=21, zero_frac=0.1)
    wl2 = W.make_random(10, 900, seed=22, zero_frac=0.4)
    plan = B.plan_for(wl1, 3)
    plan.alloc_workspace()
    for wl in (wl1, wl2, wl1):
        plan.update_counts(wl.sendcounts, wl.sdispls, wl.rdispls, wl.sendbase, wl.recvbase)
        plan.alloc_workspace()
        send, recv = wl.make_send("cuda"), wl.make_recv("cuda", fill=CANARY)
        for _ in range(2):                       # re-runnable with the same plan
            recv.fill_(CANARY)
            plan.alltoallv(send, recv)
            torch.cuda.synchronize()
            ref, rounds, _, _ = oracle_flat(wl, 3)
            assert np.array_equal(recv.cpu().numpy(), ref)
        check_rounds(plan, rounds)


@pytest.mark.parametrize("P", [10, 1100])
def test_rejected_update_leaves_the_plan_as_it_was(P):
    """New counts with a negative entry are refused; the plan still checks calls against,
    and exchanges, the counts it had.  P = 1100 takes the threaded host pass."""
    wl = W.make_random(P, 40 if P > 100 else 400, seed=31, zero_frac=0.2, gaps=P < 100)
    plan = B.plan_for(wl, 4)
    plan.alloc_workspace()
    bad = wl.sendcounts.copy()
    bad[P - 1, P // 2] = -3
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        plan.update_counts(bad, wl.sdispls, wl.rdispls, wl.sendbase, wl.recvbase)
    bad_d = wl.rdispls.copy()
    bad_d[P // 3, P - 1] = -1
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        plan.update_counts(wl.sendcounts, wl.sdispls, bad_d, wl.sendbase, wl.recvbase)
    send, recv = wl.make_send("cuda"), wl.make_recv("cuda", fill=CANARY)
    plan.alltoallv(send, recv, sendcounts=wl.sendcounts, sdispls=wl.sdispls,
                   recvcounts=wl.recvcounts, rdispls=wl.rdispls)
    torch.cuda.synchronize()
    assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl))
    other = wl.sendcounts.copy()
    other[0, 0] += 1
    with pytest.raises(B.TunaError, match="COUNT_MISMATCH"):
        plan.alltoallv(send, recv, sendcounts=other)
    # extents and payload from the threaded pass agree with the generator's
    se, re_, payload = plan.extents()
    assert (se, re_) == (wl.send_bytes, wl.recv_bytes) and payload == wl.payload_bytes_total


@pytest.mark.parametrize("kw", [dict(radix=3), dict(radix=2, flags=B.FLAG_CLASSIC_ROTATE),
                                dict(radix=2, l=4, g=3, radix_global=3), dict(radix=4, l=4, g=3, block_count=5),
                                dict(radix=12, direct=True)])
def test_update_counts_from_device_memory(kw):
    """Counts that live on the GPU (packed layout worked out there): every schedule
    must give what the oracle gives for those counts, and the plan's extents, payload
    and per-round byte counts must be those of the new counts."""
    kw = dict(kw)
    direct = kw.pop("direct", False)
    first = W.make_random(12, 300, seed=61, zero_frac=0.1)
    plan = B.plan_for(first, explicit_layout=False, **kw)
    for seed, top, zf in ((62, 900, 0.4), (63, 17, 0.0), (64, 5000, 0.8)):
        wl = W.make_random(12, top, seed=seed, zero_frac=zf)      # packed, like the device layout
        d_counts = torch.from_numpy(wl.sendcounts).cuda()
        plan.update_counts_device(d_counts)
        d_counts.fill_(-7)                                        # the plan kept its own copy
        plan.alloc_workspace()
        assert plan.extents() == (wl.send_bytes, wl.recv_bytes, wl.payload_bytes_total)
        send, recv = wl.make_send("cuda"), wl.make_recv("cuda", fill=CANARY)
        (plan.direct_alltoallv if direct else plan.alltoallv)(send, recv)
        torch.cuda.synchronize()
        assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl))
        if not direct and "l" not in kw:
            _, rounds, _, _ = oracle_flat(wl, kw["radix"])
            check_rounds(plan, rounds)
        # arrays given at call time are still compared with the plan's (fetched from the device)
        recv.fill_(CANARY)
        (plan.direct_alltoallv if direct else plan.alltoallv)(
            send, recv, sendcounts=wl.sendcounts, sdispls=wl.sdispls, recvcounts=wl.recvcounts, rdispls=wl.rdispls)
        torch.cuda.synchronize()
        assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl))
        other = wl.sendcounts.copy()
        other[3, 4] += 1
        with pytest.raises(B.TunaError, match="COUNT_MISMATCH"):
            plan.alltoallv(send, recv, sendcounts=other)
    # and back to counts from the host, with gaps
    wl = W.make_random(12, 200, seed=65, zero_frac=0.3, gaps=True)
    plan.update_counts(wl.sendcounts, wl.sdispls, wl.rdispls, wl.sendbase, wl.recvbase)
    plan.alloc_workspace()
    send, recv = wl.make_send("cuda"), wl.make_recv("cuda", fill=CANARY)
    (plan.direct_alltoallv if direct else plan.alltoallv)(send, recv)
    torch.cuda.synchronize()
    assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl))
    # device counts once more: the host update moved the plan's count buffer, so the
    # captured plan kernels are captured afresh
    wl = W.make_random(12, 333, seed=66, zero_frac=0.2)
    for _ in range(2):
        plan.update_counts_device(torch.from_numpy(wl.sendcounts).cuda())
        plan.alloc_workspace()
        send, recv = wl.make_send("cuda"), wl.make_recv("cuda", fill=CANARY)
        (plan.direct_alltoallv if direct else plan.alltoallv)(send, recv)
        torch.cuda.synchronize()
        assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl))


def test_update_waits_for_the_plans_own_exchange_in_flight():
    """An update issued on another stream while the plan's exchange is still running must
    not disturb that exchange (the library waits for it before it rewrites the tables)."""
    big = W.make_random(48, 1 << 20, seed=81, zero_frac=0.1)       # about 1 GB: a millisecond of exchange
    small = W.make_random(48, 64, seed=82, zero_frac=0.5)
    plan = B.plan_for(big, 48, explicit_layout=False)
    send, recv = big.make_send("cuda"), big.make_recv("cuda", fill=CANARY)
    d_small = torch.from_numpy(small.sendcounts).cuda()
    s_x, s_p = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    torch.cuda.synchronize()
    plan.alltoallv(send, recv, stream=s_x)
    plan.update_counts_device(d_small, stream=s_p)                   # while the exchange runs
    torch.cuda.synchronize()
    ref_plan = B.plan_for(big, 48, explicit_layout=False)            # the same exchange, undisturbed
    want = big.make_recv("cuda", fill=CANARY)
    ref_plan.alltoallv(send, want)
    torch.cuda.synchronize()
    assert torch.equal(recv, want)
    rng = np.random.default_rng(83)                                  # and pinned to the definition on samples
    s_, d_ = rng.integers(0, 48, 4096), rng.integers(0, 48, 4096)
    k_ = (rng.random(4096) * big.sendcounts[s_, d_]).astype(np.int64)
    src = torch.from_numpy(big.sendbase[s_] + big.sdispls[s_, d_] + k_).cuda()
    dst = torch.from_numpy(big.recvbase[d_] + big.rdispls[d_, s_] + k_).cuda()
    ok = torch.from_numpy(big.sendcounts[s_, d_] > 0).cuda()
    assert torch.equal(recv[dst][ok], send[src][ok])
    send2, recv2 = small.make_send("cuda"), small.make_recv("cuda", fill=CANARY)
    plan.alltoallv(send2, recv2)
    torch.cuda.synchronize()
    assert np.array_equal(recv2.cpu().numpy(), oracle_brute(small))


def test_plans_without_a_direct_list():
    """TUNA_FLAG_NO_DIRECT: the plan's own schedule works as ever, the direct exchange is
    refused, except where the single phase's lists are the direct exchange anyway."""
    wl = W.make_random(12, 300, seed=73, zero_frac=0.2, gaps=True)
    ref = oracle_brute(wl)
    send = wl.make_send("cuda")
    for kw in (dict(radix=2), dict(radix=3, l=4, g=3, radix_global=3), dict(radix=2, flags=B.FLAG_CLASSIC_ROTATE)):
        kw = dict(kw)
        kw["flags"] = kw.get("flags", 0) | B.FLAG_NO_DIRECT
        plan = B.plan_for(wl, **kw)
        plan.alloc_workspace()
        assert plan.phase_info(-2)["entries"] == 0
        recv = wl.make_recv("cuda", fill=CANARY)
        plan.alltoallv(send, recv)
        torch.cuda.synchronize()
        assert np.array_equal(recv.cpu().numpy(), ref)
        recv = wl.make_recv("cuda", fill=CANARY)
        with pytest.raises(B.TunaError, match="INVALID_ARG"):
            plan.direct_alltoallv(send, recv)
        torch.cuda.synchronize()
        assert bool((recv == CANARY).all())
    plan = B.plan_for(wl, 12, flags=B.FLAG_NO_DIRECT)   # radix >= P: the phase's lists serve
    recv = wl.make_recv("cuda", fill=CANARY)
    plan.direct_alltoallv(send, recv)
    torch.cuda.synchronize()
    assert np.array_equal(recv.cpu().numpy(), ref)
    # packed counts from device memory on a hierarchical plan without a direct list
    wp = W.make_random(12, 500, seed=74, zero_frac=0.3)
    plan = B.plan_for(W.make_uniform(12, 2), 4, l=4, g=3, radix_global=3, flags=B.FLAG_NO_DIRECT, explicit_layout=False)
    for _ in range(2):
        plan.update_counts_device(torch.from_numpy(wp.sendcounts).cuda())
        plan.alloc_workspace()
        recv = wp.make_recv("cuda", fill=CANARY)
        plan.alltoallv(wp.make_send("cuda"), recv)
        torch.cuda.synchronize()
        assert np.array_equal(recv.cpu().numpy(), oracle_brute(wp))


def test_negative_device_counts_are_refused_and_the_plan_recovers():
    wl = W.make_random(9, 300, seed=71, zero_frac=0.2)
    plan = B.plan_for(wl, 3, explicit_layout=False)
    plan.alloc_workspace()
    bad = wl.sendcounts.copy()
    bad[8, 2] = -1
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        plan.update_counts_device(torch.from_numpy(bad).cuda())
    send, recv = wl.make_send("cuda"), wl.make_recv("cuda", fill=CANARY)
    with pytest.raises(B.TunaError, match="INTERNAL"):             # its tables were rewritten
        plan.alltoallv(send, recv)
    with pytest.raises(B.TunaError, match="INTERNAL"):
        plan.direct_alltoallv(send, recv)
    torch.cuda.synchronize()
    assert bool((recv == CANARY).all())                            # nothing was moved
    plan.update_counts_device(torch.from_numpy(wl.sendcounts).cuda())
    plan.alloc_workspace()
    plan.alltoallv(send, recv)
    torch.cuda.synchronize()
    assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl))


def test_device_counts_at_p2048_match_the_host_path():
    """c5's count matrix (4.2 million pairs) through both update paths: same tables."""
    wl = W.make_c5()
    plan_h = B.plan_for(wl, wl.P, explicit_layout=False)
    plan_d = B.plan_for(W.make_uniform(wl.P, 1), wl.P, explicit_layout=False)
    plan_d.update_counts_device(torch.from_numpy(wl.sendcounts).cuda())
    assert plan_d.extents() == plan_h.extents() == (wl.send_bytes, wl.recv_bytes, wl.payload_bytes_total)
    th, td = plan_h.phase_tables(0, B.PART_DELIVER), plan_d.phase_tables(0, B.PART_DELIVER)
    for key in ("len", "pos", "src", "dst"):
        assert np.array_equal(th[key], td[key])
    send = wl.make_send("cuda")
    got = []
    for plan in (plan_h, plan_d):
        recv = wl.make_recv("cuda", fill=CANARY)
        plan.alltoallv(send, recv)
        torch.cuda.synchronize()
        got.append(recv)
    assert torch.equal(got[0], got[1])


@pytest.mark.parametrize("kw", [dict(radix=2), dict(radix=3, l=3, g=4, rg=2), dict(radix=12, direct=True)])
def test_exchange_replayed_from_a_cuda_graph(kw):
    """The exchange only enqueues kernels, so it can be captured once and replayed."""
    wl = W.make_random(12, 700, seed=41, zero_frac=0.2, gaps=True)
    kw = dict(kw)
    direct = kw.pop("direct", False)
    plan = B.plan_for(wl, kw.pop("radix"), l=kw.pop("l", None), g=kw.pop("g", 1), radix_global=kw.pop("rg", 2))
    plan.alloc_workspace()
    send, recv = wl.make_send("cuda"), wl.make_recv("cuda", fill=CANARY)
    run = plan.direct_alltoallv if direct else plan.alltoallv
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        run(send, recv)                         # warm-up outside the capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            run(send, recv)
        for _ in range(3):
            recv.copy_(wl.make_recv("cuda", fill=CANARY))
            graph.replay()
            stream.synchronize()
            assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl))
    assert plan.device_status() == 0


def test_host_buffer_entry_point():
    wl = W.make_random(9, 20000, seed=5, zero_frac=0.2, gaps=True)   # mean block over 2 KiB
    ref = oracle_brute(wl)                                   # canary 0xA5 in the gaps
    plan = B.plan_for(wl, 3)
    plan.alloc_workspace(host_staging=True)
    hs = wl.make_send().pin_memory()
    covered = np.zeros(wl.recv_bytes, dtype=bool)
    for d in range(wl.P):
        for s in range(wl.P):
            o = int(wl.recvbase[d] + wl.rdispls[d, s]) * wl.elem_size
            covered[o:o + int(wl.sendcounts[s, d]) * wl.elem_size] = True
    for schedule in (B.SCHEDULE_TUNA, B.SCHEDULE_DIRECT):
        # pinned buffers: the kernels work on host memory in place, gaps stay untouched
        hr = torch.full((wl.recv_bytes,), CANARY, dtype=torch.uint8).pin_memory()
        plan.alltoallv_host(hs, hr, schedule)
        torch.cuda.synchronize()
        assert np.array_equal(hr.numpy(), ref)
        # staged through device copies (forced, or because the memory is pageable)
        for send_h, flag in ((hs, B.HOST_STAGED), (wl.make_send(), 0)):
            hr2 = torch.zeros(wl.recv_bytes, dtype=torch.uint8)
            if flag:
                hr2 = hr2.pin_memory()
            plan.alltoallv_host(send_h, hr2, schedule | flag)
            torch.cuda.synchronize()
            assert np.array_equal(hr2.numpy()[covered], ref[covered])
    small = B.plan_for(wl, 3)
    small.alloc_workspace(host_staging=False)
    hr = torch.full((wl.recv_bytes,), CANARY, dtype=torch.uint8).pin_memory()
    small.alltoallv_host(hs, hr, B.SCHEDULE_TUNA)            # in place: no staging space needed
    torch.cuda.synchronize()
    assert np.array_equal(hr.numpy(), ref)
    with pytest.raises(B.TunaError, match="WORKSPACE"):
        small.alltoallv_host(hs, hr, B.SCHEDULE_TUNA | B.HOST_STAGED)
    with pytest.raises(B.TunaError, match="OVERLAP"):
        small.alltoallv_host(hs, hs, B.SCHEDULE_TUNA)


def test_degenerate_inputs():
    for P in (1, 2, 7):
        z = W._finish("zeros", P, 4, 1, np.zeros((P, P), dtype=np.int64))
        got, plan = gpu_run(z, 2)
        assert got.size == 0 and plan.last_launches() == 0
        one = np.zeros((P, P), dtype=np.int64)
        one[P - 1, 0] = 123457
        wl = W._finish("one", P, 1, 1, one)
        got, _ = gpu_run(wl, 2)
        assert np.array_equal(got, oracle_brute(wl))
        rc = W.make_random(P, 60, seed=9).sendcounts.copy()
        rc[0, :] = 0
        rc[:, P - 1] = 0
        wl = W._finish("rc", P, 1, 1, rc)
        for r in (2, max(2, P)):
            got, _ = gpu_run(wl, r)
            assert np.array_equal(got, oracle_brute(wl))


def test_degenerate_inputs_from_device_counts():
    """The same corner cases through the device-count update (captured plan kernels):
    one rank, two ranks, nothing to move, a single block, then real counts again."""
    for P in (1, 2, 7):
        for radix in (2, max(2, P)):
            plan = B.plan_for(W.make_uniform(P, 3), radix, explicit_layout=False)
            zeros = torch.zeros((P, P), dtype=torch.int64, device="cuda")
            for _ in range(2):                                   # the second update replays the graph
                plan.update_counts_device(zeros)
                assert plan.extents() == (0, 0, 0)
                empty = torch.empty(0, dtype=torch.uint8, device="cuda")
                plan.alltoallv(empty, empty)
                assert plan.last_launches() == 0
            one = np.zeros((P, P), dtype=np.int64)
            one[P - 1, 0] = 54321
            for counts in (one, W.make_random(P, 70, seed=3 + P).sendcounts):
                wl = W._finish("dev", P, 1, 5, counts)
                plan.update_counts_device(torch.from_numpy(wl.sendcounts).cuda())
                plan.alloc_workspace()
                send, recv = wl.make_send("cuda"), wl.make_recv("cuda", fill=CANARY)
                plan.alltoallv(send, recv)
                torch.cuda.synchronize()
                assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl))
                recv.fill_(CANARY)
                plan.direct_alltoallv(send, recv)
                torch.cuda.synchronize()
                assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl))
            plan.destroy()


# ---------------------------------------------------------------- the five workloads

def test_c1_full():
    wl = W.make_c1()
    ref, rounds, _, _ = oracle_flat(wl, 2)
    got, plan = gpu_run(wl, 2)
    assert np.array_equal(got, ref)
    check_rounds(plan, rounds)
    v = got.view(np.int32)
    for d in range(wl.P):                       # the payload names its own home
        lo, hi = int(wl.recvbase[d]), int(wl.recvbase[d] + wl.recvcounts[d].sum())
        assert np.all(((v[lo:hi] >> 10) & 1023) == d)


@pytest.mark.parametrize("r", [2, 4, 8, 16, 64])
def test_c2_full(r):
    wl = W.make_c2()
    ref, rounds, _, _ = oracle_flat(wl, r)
    for flags in (0, B.FLAG_CLASSIC_ROTATE):
        got, plan = gpu_run(wl, r, flags=flags)
        assert np.array_equal(got, ref)
    check_rounds(plan, rounds)
    got, _ = gpu_run(wl, r, direct=True)
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("rl,rg", list(itertools.product((2, 4, 16), (2, 4, 16))))
def test_c3_full(rl, rg):
    wl = W.make_c3()
    ref, rounds, _, _ = oracle_hier(wl, 16, 16, rl, rg)
    got, plan = gpu_run(wl, rl, l=16, g=16, rg=rg)
    assert np.array_equal(got, ref)
    check_rounds(plan, rounds)


@pytest.mark.parametrize("skew", [False, True])
def test_c4_scaled_down(skew):
    """The token-dispatch shape with fewer tokens and a narrower hidden size, so
    that the oracle finishes in seconds; blocks still span many chunks.  ``skew``:
    one bias per destination shared by all ranks, so a few experts draw most tokens."""
    wl = W.make_c4(P=64, tokens=256, hidden=512, skew=skew)
    if skew:
        col = wl.sendcounts.sum(axis=0)
        assert col.max() > 4 * np.median(col)                 # the hot experts really are hot
    for r in (2, 8, 64):
        ref, rounds, _, _ = oracle_flat(wl, r)
        got, plan = gpu_run(wl, r)
        assert np.array_equal(got, ref)
        check_rounds(plan, rounds)
    got, _ = gpu_run(wl, 2, direct=True)
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("r", [2, 8, 32, 2048])
def test_c5_full_flat(r):
    wl = W.make_c5()
    ref, rounds, _, _ = oracle_flat(wl, r)
    got, plan = gpu_run(wl, r, pass_args=False)
    assert np.array_equal(got, ref)
    check_rounds(plan, rounds)


def test_c5_full_hier_and_direct():
    wl = W.make_c5()
    ref, rounds, _, _ = oracle_hier(wl, 32, 64, 32, 64)
    got, plan = gpu_run(wl, 32, l=32, g=64, rg=64, pass_args=False)
    assert np.array_equal(got, ref)
    check_rounds(plan, rounds)
    got, _ = gpu_run(wl, 2, direct=True, pass_args=False)
    assert np.array_equal(got, ref)


def _block_sums(buf_words, base, displs, counts, elem_words):
    """Wrapping 64-bit sum of every block's words, via one cumulative sum."""
    cs = torch.cumsum(buf_words, 0)
    cs = torch.cat([torch.zeros(1, dtype=torch.int64, device=buf_words.device), cs])
    start = torch.from_numpy(((base[:, None] + displs) * elem_words).astype(np.int64)).to(buf_words.device)
    end = start + torch.from_numpy((counts * elem_words).astype(np.int64)).to(buf_words.device)
    return cs[end] - cs[start]


def _host_memory_available():
    """Bytes of host memory this process may still take (the smaller of what the
    machine has free and what its control group allows)."""
    import psutil
    avail = psutil.virtual_memory().available
    for limit, used in (("/sys/fs/cgroup/memory.max", "/sys/fs/cgroup/memory.current"),
                        ("/sys/fs/cgroup/memory/memory.limit_in_bytes",
                         "/sys/fs/cgroup/memory/memory.usage_in_bytes")):
        try:
            lim = open(limit).read().strip()
            if lim != "max":
                avail = min(avail, int(lim) - int(open(used).read().strip()))
        except (OSError, ValueError):
            pass
    return avail


def _equal_in_slices(dev, host, step=1 << 28):
    """Device tensor against a host array of the same bytes, a slice at a time."""
    for a in range(0, dev.numel(), step):
        b = min(a + step, dev.numel())
        if not np.array_equal(dev[a:b].cpu().numpy(), host[a:b]):
            return False
    return True


def test_c4_full_size_against_the_oracle():
    """The 8 GiB token-dispatch shape, every byte: the receive buffer of the radix-64
    schedule (the configuration the benchmark times) and of the direct exchange against
    the oracle's definition of the exchange on the same send buffer, and the schedule's
    per-round table against the oracle's radix-64 run."""
    free, _ = torch.cuda.mem_get_info()
    if free < 20 * 2**30:
        pytest.skip("needs about 20 GiB of free device memory")
    if _host_memory_available() < 30 * 2**30:
        pytest.skip("needs about 30 GiB of host memory for the oracle's buffers")
    wl = W.make_c4()
    assert wl.payload_bytes_total == 8 * 2**30
    send = wl.make_send("cuda")
    send_h = send.cpu().numpy()
    ref = np.full(wl.recv_bytes, CANARY, dtype=np.uint8)
    oracle.bruteforce(wl, send_h, ref)
    plan = B.plan_for(wl, 64)
    plan.alloc_workspace()
    recv = wl.make_recv("cuda", fill=CANARY)
    plan.alltoallv(send, recv)
    torch.cuda.synchronize()
    assert _equal_in_slices(recv, ref)
    recv.fill_(CANARY)
    plan.direct_alltoallv(send, recv)
    torch.cuda.synchronize()
    assert _equal_in_slices(recv, ref)
    del recv
    flat = np.full(wl.recv_bytes, CANARY, dtype=np.uint8)
    _, rounds, _, _ = oracle.tuna_flat(wl, 64, send_h, flat)
    assert np.array_equal(flat, ref)
    check_rounds(plan, rounds)


@pytest.mark.parametrize("schedule", ["r64", "r2", "r8_classic", "direct", "skew_r64", "skew_r2"])
def test_c4_full_size(schedule):
    """The 8 GiB token-dispatch shape in the configuration the benchmark times.
    The oracle runs this size once, in a test of its own, so here the check is (a) sampled received bytes
    against the definition of the exchange applied to the generator, and (b) a
    property that holds at any size: every one of the P^2 received blocks has the
    same 64-bit word sum as the block that was sent."""
    free, _ = torch.cuda.mem_get_info()
    if free < 70 * 2**30:
        pytest.skip("needs about 70 GiB of free device memory")
    wl = W.make_c4(skew=schedule.startswith("skew"))
    assert wl.payload_bytes_total == 8 * 2**30
    send = wl.make_send("cuda")
    recv = wl.make_recv("cuda", fill=CANARY)
    kw = dict(r64=dict(radix=64), r2=dict(radix=2), r8_classic=dict(radix=8, flags=B.FLAG_CLASSIC_ROTATE),
              direct=dict(radix=64), skew_r64=dict(radix=64), skew_r2=dict(radix=2))[schedule]
    plan = B.plan_for(wl, **kw)
    plan.alloc_workspace()
    if schedule == "direct":
        plan.direct_alltoallv(send, recv)
    else:
        plan.alltoallv(send, recv)
    torch.cuda.synchronize()
    # (a) samples
    rng = np.random.default_rng(2024)
    n = 1 << 20
    pairs = np.argwhere(wl.sendcounts > 0)                    # (the skewed routing leaves some pairs empty)
    pick = pairs[rng.integers(0, len(pairs), n)]
    s, d = pick[:, 0], pick[:, 1]
    k = (rng.random(n) * (wl.sendcounts[s, d] * wl.elem_size)).astype(np.int64)
    src = torch.from_numpy((wl.sendbase[s] + wl.sdispls[s, d]) * wl.elem_size + k).cuda()
    dst = torch.from_numpy((wl.recvbase[d] + wl.rdispls[d, s]) * wl.elem_size + k).cuda()
    assert torch.equal(recv[dst], W.payload_byte_at(wl.seed, src))
    # (b) all blocks, by checksum
    ew = wl.elem_size // 8
    sent = _block_sums(send.view(torch.int64), wl.sendbase, wl.sdispls, wl.sendcounts, ew)
    got = _block_sums(recv.view(torch.int64), wl.recvbase, wl.rdispls, wl.recvcounts, ew)
    assert torch.equal(got, sent.T)
    # the schedule's byte counts: every block is moved once per non-zero digit of its offset
    if schedule != "direct":
        r = kw["radix"]
        offs = (np.arange(wl.P)[None, :] - np.arange(wl.P)[:, None]) % wl.P
        nz = np.zeros_like(offs)
        t = offs.copy()
        while t.any():
            nz += (t % r) != 0
            t //= r
        assert sum(x["bytes"] for x in plan.rounds()) == int((wl.sendcounts * nz).sum()) * wl.elem_size


@pytest.mark.parametrize("name,kw", [("normal", dict(radix=64)), ("normal", dict(radix=4096)),
                                     ("powerlaw", dict(radix=2)),
                                     ("powerlaw", dict(radix=64, l=64, g=64, radix_global=64)),
                                     ("normal", dict(radix=64, l=64, g=64, block_count=64))])
def test_paper_scale_4096_ranks(name, kw):
    """Sec. VI-C's scale: P = 4096 ranks, 16.8 million blocks of at most 1 KiB.  Too
    large for the oracle, so the received bytes are sampled against the definition of
    the exchange applied to the generator, and the schedule's byte count is checked
    against its closed form."""
    free, _ = torch.cuda.mem_get_info()
    if free < 80 * 2**30:
        pytest.skip("needs about 80 GiB of free device memory")
    wl = W.FULL[name]()
    assert wl.P == 4096
    send = wl.make_send("cuda")
    recv = wl.make_recv("cuda", fill=CANARY)
    plan = B.plan_for(wl, explicit_layout=False, **kw)
    plan.alloc_workspace()
    plan.alltoallv(send, recv)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    rng = np.random.default_rng(4096)
    n = 1 << 22
    s = rng.integers(0, wl.P, n)
    d = rng.integers(0, wl.P, n)
    k = (rng.random(n) * wl.sendcounts[s, d]).astype(np.int64)
    ok = wl.sendcounts[s, d] > 0
    s, d, k = s[ok], d[ok], k[ok]
    src = torch.from_numpy(wl.sendbase[s] + wl.sdispls[s, d] + k).cuda()
    dst = torch.from_numpy(wl.recvbase[d] + wl.rdispls[d, s] + k).cuda()
    assert torch.equal(recv[dst], W.payload_byte_at(wl.seed, src))
    # first and last byte of every block of a few receivers
    for rank in (0, 1777, 4095):
        c = wl.sendcounts[:, rank]
        nz = np.nonzero(c)[0]
        for kk in (np.zeros_like(nz), c[nz] - 1):
            src = torch.from_numpy(wl.sendbase[nz] + wl.sdispls[nz, rank] + kk).cuda()
            dst = torch.from_numpy(wl.recvbase[rank] + wl.rdispls[rank, nz] + kk).cuda()
            assert torch.equal(recv[dst], W.payload_byte_at(wl.seed, src))
    # bytes moved: once per non-zero digit of the block's offset(s)
    if "block_count" not in kw:
        Q, N = (kw["l"], kw["g"]) if "l" in kw else (wl.P, 1)
        idx = np.arange(wl.P)
        jo = (idx[None, :] % Q - idx[:, None] % Q) % Q
        io = (idx[None, :] // Q - idx[:, None] // Q) % N
        hops = np.zeros((wl.P, wl.P), dtype=np.int64)
        for t, r in ((jo, kw["radix"]), (io, kw.get("radix_global", 2))):
            t = t.copy()
            while t.any():
                hops += (t % r) != 0
                t //= r
        assert sum(x["bytes"] for x in plan.rounds()) == int((wl.sendcounts * hops).sum())


@pytest.mark.parametrize("name", ["normal", "powerlaw", "fft_n1", "fft_n2"])
def test_paper_count_patterns(name):
    """Normal and power-law block sizes and the two FFT transposes, at P = 512."""
    wl = W.FULL[name](P=512)
    ref, rounds, _, _ = oracle_flat(wl, 8)
    got, plan = gpu_run(wl, 8, pass_args=False)
    assert np.array_equal(got, ref)
    check_rounds(plan, rounds)
    ref_h, rounds_h, _, _ = oracle_hier(wl, 32, 16, 32, 16)
    got, plan = gpu_run(wl, 32, l=32, g=16, rg=16, pass_args=False)
    assert np.array_equal(got, ref_h) and np.array_equal(ref_h, ref)
    check_rounds(plan, rounds_h)
    got, _ = gpu_run(wl, 2, direct=True, pass_args=False)
    assert np.array_equal(got, ref)


def test_block_larger_than_4_gib():
    """64-bit offsets end to end: one block of 5 GiB + 3 bytes (larger than any 32-bit
    count or displacement), next to small unaligned ones, through a two-hop schedule."""
    free, _ = torch.cuda.mem_get_info()
    if free < 30 * 2**30:
        pytest.skip("needs about 30 GiB of free device memory")
    counts = np.array([[5, 7, 0, 11], [13, 0, 17, 19], [0, 23, 29, 31], [37, 41, 43, 0]], dtype=np.int64)
    counts[1, 0] = 5 * 2**30 + 3
    wl = W._finish("huge", 4, 1, 99, counts)
    send = wl.make_send("cuda")
    for kw, direct in ((dict(radix=2), False), (dict(radix=2, flags=B.FLAG_CLASSIC_ROTATE), False),
                       (dict(radix=4), True)):
        recv = wl.make_recv("cuda", fill=CANARY)
        plan = B.plan_for(wl, **kw)
        plan.alloc_workspace()
        (plan.direct_alltoallv if direct else plan.alltoallv)(send, recv)
        torch.cuda.synchronize()
        for s in range(4):
            for d in range(4):
                n = int(wl.sendcounts[s, d])
                a = int(wl.sendbase[s] + wl.sdispls[s, d])
                b = int(wl.recvbase[d] + wl.rdispls[d, s])
                assert torch.equal(recv[b:b + n], send[a:a + n]), (s, d)
        assert int(wl.recv_bytes) == int(counts.sum())     # packed: every byte is covered
        plan.set_workspace(None)
        plan.destroy()
        del recv
        torch.cuda.empty_cache()


def test_random_configurations():
    """Seeded sweep over rank counts, groupings, radices, element sizes, sparsity,
    layouts with gaps, buffer misalignment and both placement modes."""
    rng = np.random.default_rng(20241102)
    for case in range(90):
        P = int(rng.integers(1, 49))
        divs = [d for d in range(1, P + 1) if P % d == 0]
        l = int(rng.choice(divs))
        g = P // l
        r = int(rng.integers(2, max(2, l) + 1))
        rg = int(rng.integers(2, max(2, g) + 1))
        elem = int(rng.choice([1, 2, 3, 4, 8]))
        maxc = int(rng.choice([0, 1, 17, 300, 5000]))
        wl = W.make_random(P, maxc, elem_size=elem, seed=1000 + case,
                           zero_frac=float(rng.choice([0.0, 0.3, 0.9])), gaps=bool(rng.integers(0, 2)))
        flags = int(rng.choice([0, B.FLAG_CLASSIC_ROTATE, B.FLAG_BULK_COPY]))
        mis = int(rng.choice([0, 0, 1, 5, 8]))
        ref = oracle_brute(wl)
        got, plan = gpu_run(wl, r, l=l, g=g, rg=rg, flags=flags, misalign=mis,
                            explicit=True)
        assert np.array_equal(got, ref), (case, P, l, g, r, rg, elem, maxc, flags, mis)
        assert plan.device_status() == 0
        if g == 1:
            _, rounds, _, _ = oracle_flat(wl, r)
        else:
            _, rounds, _, _ = oracle_hier(wl, l, g, r, rg)
        check_rounds(plan, rounds)


# ---------------------------------------------------------------- staggered inter-group exchange

def oracle_staggered(wl, Q, N, rl, bc):
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    return oracle.tuna_hier_staggered(wl, Q, N, rl, bc, send, recv)


STAGGERED = [(Q, N, rl, bc) for Q, N in [(1, 5), (5, 1), (2, 2), (3, 4), (4, 3), (8, 4), (16, 16)]
             for rl in sorted({2, max(2, Q)})
             for bc in sorted({1, 3, Q, Q + 1, Q * N, 2 * Q * N})]


@pytest.mark.parametrize("Q,N,rl,bc", STAGGERED)
def test_staggered_small(Q, N, rl, bc):
    """Algorithm 2: result, the Q(N-1) steps with their bytes, one launch per batch."""
    P = Q * N
    wl = W.make_random(P, 300, elem_size=1, seed=3000 + P + bc, zero_frac=0.25, gaps=True)
    ref, rounds, (Kl, Kg), batches = oracle_staggered(wl, Q, N, rl, bc)
    got, plan = gpu_run(wl, rl, l=Q, g=N, block_count=bc, misalign=(bc % 3) * 5)
    assert np.array_equal(got, ref)
    check_rounds(plan, rounds)
    assert plan.device_status() == 0
    local_phases = sum(1 for f in range(plan.num_phases()) if plan.phase_info(f, B.PART_KEEP)["level"] == 0)
    assert plan.num_phases() - local_phases == batches
    # every batch is a launch of its own unless it moves no bytes at all
    assert plan.last_launches() <= local_phases + batches
    if wl.sendcounts.min() > 0:
        assert plan.last_launches() == local_phases + batches


def test_staggered_rejects_bad_arguments():
    wl = W.make_random(12, 10, seed=5)
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        B.plan_for(wl, 2, l=4, g=3, block_count=-1)
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        B.plan_for(wl, 2, l=4, g=3, block_count=2, flags=B.FLAG_CLASSIC_ROTATE)
    with pytest.raises(B.TunaError, match="BAD_HIERARCHY"):
        B.plan_for(wl, 2, l=5, g=3, block_count=2)


def test_staggered_update_counts_and_full_c3():
    """New counts on a staggered plan; then the 16 x 16 Zipf configuration at full size."""
    wl = W.make_random(12, 200, seed=8, gaps=True)
    plan = B.plan_for(wl, 2, l=4, g=3, block_count=4)
    wl2 = W.make_random(12, 500, seed=9, zero_frac=0.5, gaps=True)
    plan.update_counts(wl2.sendcounts, wl2.sdispls, wl2.rdispls, wl2.sendbase, wl2.recvbase)
    plan.alloc_workspace()
    send = wl2.make_send("cuda")
    recv = wl2.make_recv("cuda", fill=CANARY)
    plan.alltoallv(send, recv)
    torch.cuda.synchronize()
    assert np.array_equal(recv.cpu().numpy(), oracle_brute(wl2))
    c3 = W.make_c3()
    ref, rounds, _, batches = oracle_staggered(c3, 16, 16, 16, 16)
    got, plan3 = gpu_run(c3, 16, l=16, g=16, block_count=16)
    assert np.array_equal(got, ref)
    check_rounds(plan3, rounds)


# ---------------------------------------------------------------- rows with gather / scatter maps

def _rows_inputs(wl, seed, identity_gather=False, identity_scatter=False):
    rb = wl.elem_size
    rng = np.random.default_rng(seed)
    send_rows, recv_rows = wl.send_bytes // rb, wl.recv_bytes // rb
    in_rows = send_rows + (0 if identity_gather else 7)
    out_rows = recv_rows + (0 if identity_scatter else 5)
    gather = None if identity_gather else rng.integers(0, in_rows, send_rows)
    scatter = None if identity_scatter else rng.permutation(out_rows)[:recv_rows]
    rows_in = rng.integers(0, 256, (max(in_rows, 1), rb), dtype=np.uint8)[:in_rows]
    return gather, scatter, rows_in, out_rows


def _rows_gpu(wl, gather, scatter, rows_in, out_rows):
    rb = wl.elem_size
    plan = B.plan_for(wl, 2)
    dev = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()
    d_in = torch.from_numpy(rows_in).cuda()
    d_out = torch.full((out_rows, rb), CANARY, dtype=torch.uint8, device="cuda")
    plan.set_row_maps(dev(gather), dev(scatter), rows_in.shape[0], out_rows)
    plan.rows_alltoallv(d_in, d_out)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    return d_out.cpu().numpy(), plan


@pytest.mark.parametrize("P,maxc,rb,gaps", [(1, 5, 16, False), (5, 9, 3, True), (8, 40, 16, False),
                                            (12, 30, 40, True), (33, 20, 264, False),
                                            (16, 12, 8192, False), (64, 3, 100, True)])
@pytest.mark.parametrize("ident", [(False, False), (True, False), (False, True), (True, True)])
def test_rows_exchange(P, maxc, rb, gaps, ident):
    wl = W.make_random(P, maxc, elem_size=rb, seed=60 + P, zero_frac=0.2, gaps=gaps)
    gather, scatter, rows_in, out_rows = _rows_inputs(wl, 7 * P + rb, *ident)
    ref = np.full((out_rows, rb), CANARY, dtype=np.uint8)
    oracle.rows_alltoallv(wl, gather, scatter, rows_in, ref)
    got, plan = _rows_gpu(wl, gather, scatter, rows_in, out_rows)
    assert np.array_equal(got, ref)
    assert plan.last_launches() == (1 if wl.payload_bytes_total else 0)


def test_rows_exchange_errors_and_recount():
    wl = W.make_random(6, 10, elem_size=32, seed=2, gaps=False)
    gather, scatter, rows_in, out_rows = _rows_inputs(wl, 5)
    plan = B.plan_for(wl, 2)
    d_in = torch.from_numpy(rows_in).cuda()
    d_out = torch.full((out_rows, 32), CANARY, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.TunaError, match="COUNT_MISMATCH"):      # no maps yet
        plan.rows_alltoallv(d_in, d_out)
    s0, d0 = (int(v[0]) for v in np.nonzero(wl.sendcounts))       # a pair that exchanges rows
    bad = gather.copy()
    bad[wl.sdispls[s0, d0] + wl.sendbase[s0]] = rows_in.shape[0]  # one row past the end of rows_in
    with pytest.raises(B.TunaError, match="RANGE"):
        plan.set_row_maps(torch.from_numpy(bad).cuda(), torch.from_numpy(scatter).cuda(),
                          rows_in.shape[0], out_rows)
    bad = scatter.copy()
    bad[wl.rdispls[d0, s0] + wl.recvbase[d0]] = -1
    with pytest.raises(B.TunaError, match="RANGE"):
        plan.set_row_maps(torch.from_numpy(gather).cuda(), torch.from_numpy(bad).cuda(),
                          rows_in.shape[0], out_rows)
    with pytest.raises(B.TunaError, match="COUNT_MISMATCH"):      # the failed call left no maps behind
        plan.rows_alltoallv(d_in, d_out)
    plan.set_row_maps(torch.from_numpy(gather).cuda(), torch.from_numpy(scatter).cuda(),
                      rows_in.shape[0], out_rows)
    with pytest.raises(B.TunaError, match="OVERLAP"):
        plan.rows_alltoallv(d_in, d_in)
    plan.rows_alltoallv(d_in, d_out)
    torch.cuda.synchronize()
    # new counts invalidate the maps
    wl2 = W.make_random(6, 14, elem_size=32, seed=3)
    plan.update_counts(wl2.sendcounts, wl2.sdispls, wl2.rdispls, wl2.sendbase, wl2.recvbase)
    with pytest.raises(B.TunaError, match="COUNT_MISMATCH"):
        plan.rows_alltoallv(d_in, d_out)
    g2, s2, in2, out2 = _rows_inputs(wl2, 9)
    ref = np.full((out2, 32), CANARY, dtype=np.uint8)
    oracle.rows_alltoallv(wl2, g2, s2, in2, ref)
    d_in2 = torch.from_numpy(in2).cuda()
    d_out2 = torch.full((out2, 32), CANARY, dtype=torch.uint8, device="cuda")
    plan.set_row_maps(torch.from_numpy(g2).cuda(), torch.from_numpy(s2).cuda(), in2.shape[0], out2)
    plan.rows_alltoallv(d_in2, d_out2)
    torch.cuda.synchronize()
    assert np.array_equal(d_out2.cpu().numpy(), ref)


def test_rows_exchange_token_dispatch():
    """The token-dispatch shape, scaled down: P = 64 ranks, 256 tokens of 1 KiB per
    rank, top-2 routing; tokens leave in token order and arrive in expert order."""
    P, tokens, hidden = 64, 256, 512
    wl = W.make_c4(P=P, tokens=tokens, hidden=hidden)
    first, second = W.moe_top2_routing(wl.seed, P, tokens)
    gather, scatter = W.moe_row_maps(first, second)
    rng = np.random.default_rng(11)
    rows_in = rng.integers(0, 256, (P * tokens, wl.elem_size), dtype=np.uint8)
    ref = np.full((2 * P * tokens, wl.elem_size), CANARY, dtype=np.uint8)
    oracle.rows_alltoallv(wl, gather, scatter, rows_in, ref)
    plan = B.plan_for(wl, 64, explicit_layout=False)
    d_in = torch.from_numpy(rows_in).cuda()
    d_out = torch.full(ref.shape, CANARY, dtype=torch.uint8, device="cuda")
    plan.set_row_maps(torch.from_numpy(gather).cuda(), torch.from_numpy(scatter).cuda(),
                      rows_in.shape[0], ref.shape[0])
    plan.rows_alltoallv(d_in, d_out)
    torch.cuda.synchronize()
    assert np.array_equal(d_out.cpu().numpy(), ref)
    # the unfused route gives the same rows: gather, exchange, scatter
    send = d_in[torch.from_numpy(gather).cuda()].contiguous()
    recv = torch.empty_like(send)
    plan.direct_alltoallv(send, recv)
    out2 = torch.full(ref.shape, CANARY, dtype=torch.uint8, device="cuda")
    out2[torch.from_numpy(scatter).cuda()] = recv
    torch.cuda.synchronize()
    assert torch.equal(out2, d_out)

"""Pins for the CPU oracle: values the paper prints, closed forms, the
definition of the exchange, and reductions to simpler cases.  No GPU."""
import itertools
import math

import numpy as np
import pytest

import oracle
from conftest import read_golden
from paper_2411_02581_b200 import workloads as W

CANARY = 0xA5


def run_flat(wl, r, trace_rank=-1):
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    return (send,) + oracle.tuna_flat(wl, r, send, recv, trace_rank)


def brute(wl):
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    return oracle.bruteforce(wl, send, recv)


def digits(o, r, w):
    return [(o // r ** x) % r for x in range(w)]


def nnz(o, r):
    n = 0
    while o:
        n += (o % r) != 0
        o //= r
    return n


def closed_form_K(P, r):
    """Non-empty rounds: all (r-1) digit values below the top digit position,
    plus the values the top digit can take for offsets below P."""
    if P == 1:
        return 0
    w = 0
    while r ** w < P:
        w += 1
    return (w - 1) * (r - 1) + (P - 1) // r ** (w - 1)


# ---------------------------------------------------------------- definition

def test_bruteforce_self_describing_payload():
    """Every received element names (src, dst, idx); the definition of the
    exchange says which triple must sit where."""
    wl = W.make_c1()
    recv = brute(wl).view(np.int32)
    seen = 0
    for d in range(wl.P):
        for s in range(wl.P):
            c = int(wl.sendcounts[s, d])
            o = int(wl.recvbase[d] + wl.rdispls[d, s])
            got = recv[o:o + c]
            assert np.array_equal(got >> 20, np.full(c, s))
            assert np.array_equal((got >> 10) & 1023, np.full(c, d))
            assert np.array_equal(got & 1023, np.arange(c))
            seen += c
    assert seen == wl.sendcounts.sum() == recv.size


def test_bruteforce_leaves_gaps_untouched():
    wl = W.make_random(9, 40, elem_size=2, seed=3, gaps=True)
    recv = brute(wl)
    covered = np.zeros(wl.recv_bytes, dtype=bool)
    for d in range(wl.P):
        for s in range(wl.P):
            o = int(wl.recvbase[d] + wl.rdispls[d, s]) * wl.elem_size
            covered[o:o + int(wl.sendcounts[s, d]) * wl.elem_size] = True
    assert (~covered).sum() > 0
    assert np.all(recv[~covered] == CANARY)


# ---------------------------------------------------------------- schedule shape

def test_round_counts_printed_values():
    g = read_golden("round_counts.txt")
    for P, K in zip(map(int, g["bruck_P"].split()), map(int, g["bruck_K"].split())):
        assert len(oracle.round_list(P, 2)) == K == int(math.log2(P))
    for P in (2, 3, 8, 15, 64):
        assert len(oracle.round_list(P, P)) == P - 1      # spread-out end


@pytest.mark.parametrize("P", list(range(1, 41)) + [64, 100, 255, 256, 257, 2048])
def test_round_count_bound_and_closed_form(P):
    for r in sorted(set(list(range(2, min(P, 40) + 1)) + [max(2, P)])):
        rl = oracle.round_list(P, r)
        w = oracle.num_digits(P, r)
        assert r ** w >= P and (w == 0 or r ** (w - 1) < P)
        assert len(rl) <= w * (r - 1)                     # the paper's bound
        assert len(rl) == closed_form_K(P, r)
        if r ** w == P:
            assert len(rl) == w * (r - 1)                 # bound is tight for P = r^w
        assert rl == sorted(rl)                           # x outer, z inner
        dists = [z * r ** x for x, z in rl]
        assert len(set(dists)) == len(dists) and all(0 < d < P for d in dists)


def test_temp_buffer_printed_values():
    g = read_golden("temp_buffer_slots.txt")
    P = int(g["P"])
    wl = W.make_random(P, 5, seed=1)
    for r in (2, 3, 4):
        _, _, _, B, _ = run_flat(wl, r)
        assert B == int(g[f"B_r{r}"]) == P - (len(oracle.round_list(P, r)) + 1)
    assert oracle.tmap(P, 2, 3) == int(g["tmap_r2_o3"])
    assert oracle.tmap(P, 2, 5) == int(g["tmap_r2_o5"])
    for r in (7, 8):                                      # r > P - 2: no T at all
        _, _, _, B, _ = run_flat(wl, r)
        assert B == 0


@pytest.mark.parametrize("P", range(2, 41))
def test_tmap_is_a_bijection_onto_the_slots(P):
    """The map counts the direct offsets below o, so it must enumerate the
    non-direct offsets 0..B-1 in ascending order, for every radix."""
    for r in range(2, P + 1):
        K = len(oracle.round_list(P, r))
        direct = {z * r ** x for x, z in oracle.round_list(P, r)}
        assert len(direct) == K
        ts = []
        for o in range(P):
            t = oracle.tmap(P, r, o)
            if o == 0 or o in direct:
                assert t == -1
            else:
                assert t == o - 1 - sum(1 for d in direct if d < o)
                ts.append(t)
        assert ts == list(range(P - K - 1))


# ---------------------------------------------------------------- worked example

def test_fig2_worked_example():
    g = read_golden("fig2_flat_example.txt")
    P, r, rank = int(g["P"]), int(g["radix"]), int(g["rank"])
    pair = lambda s: tuple(map(int, s.split(">")))
    sent = [pair(t) for t in g["round0_send_blocks"].split()]
    meta = list(map(int, g["round0_metadata"].split()))
    counts = np.array([[1, 4, 6, 7], [2, 5, 3, 9], [8, 1, 2, 3], [4, 6, 5, 1]], dtype=np.int64)
    for (s, d), m in zip(sent, meta):
        counts[s, d] = m
    wl = W._finish("fig2", P, 1, 5, counts)
    _, recv, rounds, B, tr = run_flat(wl, r, trace_rank=rank)
    assert np.array_equal(recv, brute(wl))
    T = oracle
    r0s = tr[(tr[:, T.TR_ROUND] == 0) & (tr[:, T.TR_KIND] == 0)]
    assert set(r0s[:, T.TR_PARTNER]) == {int(g["round0_send_to"])}
    assert [(a, b) for a, b in r0s[:, [T.TR_ORIGIN, T.TR_DEST]]] == sent
    assert list(r0s[:, T.TR_BYTES]) == meta
    r0r = tr[(tr[:, T.TR_ROUND] == 0) & (tr[:, T.TR_KIND] == 1)]
    assert set(r0r[:, T.TR_PARTNER]) == {int(g["round0_recv_from"])}
    inR = [(a, b) for a, b, pl in r0r[:, [T.TR_ORIGIN, T.TR_DEST, T.TR_PLACE]] if pl == 1]
    inT = [(a, b) for a, b, pl in r0r[:, [T.TR_ORIGIN, T.TR_DEST, T.TR_PLACE]] if pl == 2]
    assert inR == [pair(g["round0_recv_into_R"])]
    assert inT == [pair(g["round0_recv_into_T"])]
    r1s = tr[(tr[:, T.TR_ROUND] == 1) & (tr[:, T.TR_KIND] == 0)]
    fromT = [(a, b) for a, b, pl in r1s[:, [T.TR_ORIGIN, T.TR_DEST, T.TR_PLACE]] if pl == 2]
    assert fromT == [pair(g["round1_forward_from_T"])]
    assert set(r1s[:, T.TR_PARTNER]) == {int(g["round1_forward_to"])}
    assert B == 1


def test_final_blocks_per_phase_and_direct_blocks():
    """A rank receives at most r^x blocks per round of digit x that have
    arrived; single-digit (direct) offsets never go through T."""
    g = read_golden("temp_buffer_slots.txt")
    T = oracle
    for P, r in [(8, 2), (8, 3), (8, 4), (27, 3), (30, 4), (17, 2)]:
        wl = W.make_random(P, 9, seed=2)
        _, _, rounds, B, tr = run_flat(wl, r, trace_rank=P // 2)
        rl = oracle.round_list(P, r)
        for k, (x, z) in enumerate(rl):
            rr = tr[(tr[:, T.TR_ROUND] == k) & (tr[:, T.TR_KIND] == 1)]
            finals = rr[rr[:, T.TR_PLACE] == 1]
            assert len(finals) <= r ** x
            if (P, r, k) == (8, 2, 1):
                assert len(finals) == int(g["final_blocks_round1_r2"])
            # the first block of every round is the direct one: offset z*r^x
            assert rr[0, T.TR_OFFSET] == z * r ** x and rr[0, T.TR_PLACE] == 1
            ss = tr[(tr[:, T.TR_ROUND] == k) & (tr[:, T.TR_KIND] == 0)]
            assert ss[0, T.TR_OFFSET] == z * r ** x and ss[0, T.TR_PLACE] == 0
            # a received block is in R exactly when it has reached its destination
            for row in rr:
                assert (row[T.TR_PLACE] == 1) == (row[T.TR_DEST] == P // 2)
            # and a block is read from S exactly when it has never moved
            for row in ss:
                assert (row[T.TR_PLACE] == 0) == (row[T.TR_ORIGIN] == P // 2)


# ---------------------------------------------------------------- result and conservation

FLAT_CASES = [(P, r) for P in (1, 2, 3, 4, 5, 7, 8, 9, 12, 16, 17) for r in range(2, max(2, P) + 1)]
FLAT_CASES += [(33, 2), (33, 6), (33, 33), (64, 4), (64, 8), (100, 10), (100, 7)]


@pytest.mark.parametrize("P,r", FLAT_CASES)
def test_flat_equals_definition_and_conserves_bytes(P, r):
    wl = W.make_random(P, 23, elem_size=3, seed=100 + P, zero_frac=0.25, gaps=True)
    _, recv, rounds, B, _ = run_flat(wl, r)
    assert np.array_equal(recv, brute(wl))
    rl = oracle.round_list(P, r)
    assert [(int(a), int(b)) for a, b in rounds[:, [oracle.RS_X, oracle.RS_Z]]] == rl
    C = wl.sendcounts * wl.elem_size
    w = oracle.num_digits(P, r)
    per_offset = np.array([sum(C[s, (s + o) % P] for s in range(P)) for o in range(P)])
    for row, (x, z) in zip(rounds, rl):
        offs = [o for o in range(P) if digits(o, r, w)[x] == z]
        assert row[oracle.RS_UNITS] == P * len(offs)
        assert len(offs) <= r ** max(w - 1, 0)
        assert row[oracle.RS_BYTES_SENT] == row[oracle.RS_BYTES_RECV] == per_offset[offs].sum()
    total = sum(int(per_offset[o]) * nnz(o, r) for o in range(P))
    assert rounds[:, oracle.RS_BYTES_SENT].sum() == total


@pytest.mark.parametrize("r,w", [(2, 3), (2, 5), (3, 2), (3, 3), (4, 2), (5, 2), (8, 2)])
def test_uniform_counts_reproduce_D(r, w):
    """Equal block sizes and P = r^w: every round carries r^(w-1) blocks per
    rank, D = w (r-1) r^(w-1) blocks in total (the uniform parameterised
    exchange the algorithm generalises)."""
    P = r ** w
    wl = W.make_uniform(P, 6, elem_size=2)
    _, recv, rounds, _, _ = run_flat(wl, r)
    assert np.array_equal(recv, brute(wl))
    assert np.all(rounds[:, oracle.RS_UNITS] == P * r ** (w - 1))
    assert rounds[:, oracle.RS_UNITS].sum() == P * w * (r - 1) * r ** (w - 1)
    assert rounds[:, oracle.RS_BYTES_SENT].sum() == 12 * P * w * (r - 1) * r ** (w - 1)


@pytest.mark.parametrize("P", [2, 5, 16, 31])
def test_radix_P_moves_every_block_once(P):
    wl = W.make_random(P, 50, seed=P)
    _, recv, rounds, B, _ = run_flat(wl, P)
    assert B == 0 and len(rounds) == P - 1
    assert np.all(rounds[:, oracle.RS_UNITS] == P)
    off_diag = wl.sendcounts.sum() - np.trace(wl.sendcounts)
    assert rounds[:, oracle.RS_BYTES_SENT].sum() == off_diag * wl.elem_size
    assert np.array_equal(recv, brute(wl))


def test_degenerate_inputs():
    for P, r in [(1, 2), (2, 2), (6, 2), (6, 3)]:
        z = W._finish("zeros", P, 4, 1, np.zeros((P, P), dtype=np.int64))
        _, recv, rounds, _, _ = run_flat(z, r)
        assert recv.size == 0 and rounds[:, oracle.RS_BYTES_SENT].sum() == 0
        one = np.zeros((P, P), dtype=np.int64)
        one[P - 1, 0] = 100000
        wl = W._finish("one", P, 1, 1, one)
        _, recv, _, _, _ = run_flat(wl, r)
        assert np.array_equal(recv, brute(wl))
        zero_row_col = W.make_random(P, 12, seed=9).sendcounts.copy()
        zero_row_col[0, :] = 0
        zero_row_col[:, P - 1] = 0
        wl = W._finish("rc", P, 1, 1, zero_row_col)
        _, recv, _, _, _ = run_flat(wl, r)
        assert np.array_equal(recv, brute(wl))


# ---------------------------------------------------------------- hierarchical

def run_hier(wl, Q, N, rl, rg, after=False):
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    return oracle.tuna_hier(wl, Q, N, rl, rg, send, recv, want_after_local=after)


def test_fig5_hier_example():
    g = read_golden("fig5_hier_example.txt")
    P, N, Q, r = int(g["P"]), int(g["N"]), int(g["Q"]), int(g["radix"])
    wl = W.make_random(P, 17, seed=15, gaps=True)
    recv, rounds, (Kl, Kg), after = run_hier(wl, Q, N, r, N, after=True)
    assert Kl == int(g["local_steps"]) and Kg == int(g["global_steps"]) == N - 1
    ref = brute(wl)
    assert np.array_equal(recv, ref)
    # after the local phase R holds exactly the blocks from ranks of the own group
    own = np.zeros(wl.recv_bytes, dtype=bool)
    for d in range(P):
        for s in range(P):
            if s // Q == d // Q:
                o = int(wl.recvbase[d] + wl.rdispls[d, s]) * wl.elem_size
                own[o:o + int(wl.sendcounts[s, d]) * wl.elem_size] = True
    assert np.array_equal(after[own], ref[own])
    assert np.all(after[~own] == CANARY)
    # coalesced rounds: every rank sends one super-block (Q blocks) per round
    gl = rounds[rounds[:, oracle.RS_LEVEL] == 1]
    assert np.all(gl[:, oracle.RS_UNITS] == P)


HIER_CASES = [(Q, N, rl, rg) for Q, N in [(1, 1), (1, 5), (5, 1), (2, 2), (3, 4), (4, 3), (5, 3),
                                          (4, 4), (6, 5), (8, 4)]
              for rl in sorted({2, 3, max(2, Q)}) if rl <= max(2, Q)
              for rg in sorted({2, 3, max(2, N)}) if rg <= max(2, N)]


@pytest.mark.parametrize("Q,N,rl,rg", HIER_CASES)
def test_hier_equals_definition_and_conserves_bytes(Q, N, rl, rg):
    P = Q * N
    wl = W.make_random(P, 19, elem_size=2, seed=7 * P + rl + rg, zero_frac=0.2, gaps=True)
    recv, rounds, (Kl, Kg), _ = run_hier(wl, Q, N, rl, rg)
    assert np.array_equal(recv, brute(wl))
    assert Kl == closed_form_K(Q, rl) and Kg == closed_form_K(N, rg)
    assert np.all(rounds[:, oracle.RS_BYTES_SENT] == rounds[:, oracle.RS_BYTES_RECV])
    C = wl.sendcounts * wl.elem_size
    loc = glo = 0
    for s in range(P):
        for d in range(P):
            loc += int(C[s, d]) * nnz((d % Q - s % Q) % Q, rl)
            glo += int(C[s, d]) * nnz((d // Q - s // Q) % N, rg)
    lv = rounds[:, oracle.RS_LEVEL]
    assert rounds[lv == 0][:, oracle.RS_BYTES_SENT].sum() == loc
    assert rounds[lv == 1][:, oracle.RS_BYTES_SENT].sum() == glo
    # per-round closed form: a local round (x, z) carries the blocks whose local
    # offset has digit x equal to z, a global round those whose group offset has
    wl_, wg_ = oracle.num_digits(Q, rl), oracle.num_digits(N, rg)
    for row in rounds:
        x, z = int(row[oracle.RS_X]), int(row[oracle.RS_Z])
        tot = 0
        for s in range(P):
            for d in range(P):
                jo, io = (d % Q - s % Q) % Q, (d // Q - s // Q) % N
                if row[oracle.RS_LEVEL] == 0 and digits(jo, rl, max(wl_, 1))[x] == z:
                    tot += int(C[s, d])
                if row[oracle.RS_LEVEL] == 1 and digits(io, rg, max(wg_, 1))[x] == z:
                    tot += int(C[s, d])
        assert row[oracle.RS_BYTES_SENT] == tot


# ---------------------------------------------------------------- staggered (Algorithm 2)

def run_staggered(wl, Q, N, rl, bc):
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    return oracle.tuna_hier_staggered(wl, Q, N, rl, bc, send, recv)


STAGGERED_CASES = [(Q, N, rl, bc) for Q, N in [(1, 1), (1, 5), (5, 1), (2, 2), (3, 4), (4, 3), (6, 5)]
                   for rl in sorted({2, max(2, Q)})
                   for bc in sorted({1, 2, Q, Q + 1, Q * N, 3 * Q * N})]


@pytest.mark.parametrize("Q,N,rl,bc", STAGGERED_CASES)
def test_staggered_equals_definition(Q, N, rl, bc):
    """Sec. IV-B (figure of the two inter-node patterns): the staggered exchange takes
    (N - 1) * Q steps of one block per rank where the coalesced one takes N - 1 of Q
    blocks; both end in the MPI_Alltoallv result."""
    P = Q * N
    wl = W.make_random(P, 23, elem_size=3, seed=11 * P + rl + bc, zero_frac=0.25, gaps=True)
    recv, rounds, (Kl, Kg), batches = run_staggered(wl, Q, N, rl, bc)
    assert np.array_equal(recv, brute(wl))
    assert Kl == closed_form_K(Q, rl) and Kg == (N - 1) * Q
    # batches of block_count consecutive step indices ii in [0, P); the first Q
    # indices name the own group and move nothing
    want_batches = sum(1 for lo in range(0, P, bc) if min(P, lo + bc) > Q)
    assert batches == want_batches
    gl = rounds[rounds[:, oracle.RS_LEVEL] == 1]
    assert len(gl) == Kg
    assert np.all(gl[:, oracle.RS_UNITS] == P)           # one block per rank per step
    assert np.all(gl[:, oracle.RS_BYTES_SENT] == gl[:, oracle.RS_BYTES_RECV])
    # step (gi, gr): every rank (n, q) receives the block that rank ((n + gi) mod N, gr)
    # owns for it
    C = wl.sendcounts * wl.elem_size
    for row in gl:
        gi, gr = int(row[oracle.RS_X]), int(row[oracle.RS_Z])
        tot = sum(int(C[((n + gi) % N) * Q + gr, n * Q + q]) for n in range(N) for q in range(Q))
        assert row[oracle.RS_BYTES_SENT] == tot
    assert [(int(a), int(b)) for a, b in gl[:, [oracle.RS_X, oracle.RS_Z]]] == \
        [(gi, gr) for gi in range(1, N) for gr in range(Q)]


@pytest.mark.parametrize("Q,N", [(3, 4), (4, 3), (2, 5)])
def test_staggered_steps_add_up_to_coalesced_rounds(Q, N):
    """The Q steps of group distance gi carry what one coalesced round carries: the
    super-blocks between groups gi apart.  Algorithm 2 sends towards (n - gi),
    Algorithm 3 towards (n + z), so distance gi matches round z = N - gi."""
    P = Q * N
    wl = W.make_random(P, 31, elem_size=1, seed=77 + P, zero_frac=0.1)
    _, rs, (Kl, _), _ = run_staggered(wl, Q, N, 2, 1)
    _, rc, (Kl2, Kg2), _ = run_hier(wl, Q, N, 2, N)
    assert Kl == Kl2 and Kg2 == N - 1
    assert np.array_equal(rs[:Kl], rc[:Kl])              # same local phase
    co = {int(r[oracle.RS_Z]): int(r[oracle.RS_BYTES_SENT]) for r in rc[Kl:]}
    for gi in range(1, N):
        steps = rs[Kl:][rs[Kl:, oracle.RS_X] == gi]
        assert steps[:, oracle.RS_BYTES_SENT].sum() == co[N - gi]


@pytest.mark.parametrize("P,r", [(6, 2), (9, 3), (16, 4), (13, 2)])
def test_hier_reduces_to_flat(P, r):
    """One group (N = 1) is the flat exchange over Q = P ranks; one rank per
    group (Q = 1) is the flat exchange over the N = P groups."""
    wl = W.make_random(P, 30, seed=P + r, gaps=True)
    _, recv_f, rounds_f, _, _ = run_flat(wl, r)
    recv_a, rounds_a, _, _ = run_hier(wl, P, 1, r, 2)
    recv_b, rounds_b, _, _ = run_hier(wl, 1, P, 2, r)
    assert np.array_equal(recv_a, recv_f) and np.array_equal(recv_b, recv_f)
    assert np.array_equal(rounds_a, rounds_f)
    assert np.array_equal(rounds_b[:, 1:], rounds_f[:, 1:])
    assert np.all(rounds_b[:, oracle.RS_LEVEL] == 1)


# ---------------------------------------------------------------- the five shapes, scaled down

def test_workload_shapes_small():
    c1 = W.make_c1()
    _, recv, _, _, _ = run_flat(c1, 2)
    assert np.array_equal(recv, brute(c1))
    c2 = W.make_c2(P=16, max_bytes=512)
    for r in (2, 4, 16):
        _, recv, _, _, _ = run_flat(c2, r)
        assert np.array_equal(recv, brute(c2))
    c3 = W.make_c3(l=4, g=4, cmax=300)
    for rl, rg in itertools.product((2, 4), (2, 4)):
        recv, _, _, _ = run_hier(c3, 4, 4, rl, rg)
        assert np.array_equal(recv, brute(c3))
    c4 = W.make_c4(P=8, tokens=64, hidden=32)
    assert c4.payload_bytes_total == 8 * 64 * 2 * 64
    for r in (2, 8):
        _, recv, _, _, _ = run_flat(c4, r)
        assert np.array_equal(recv, brute(c4))
    c5 = W.make_c5(P=64, hier=(8, 8))
    for r in (2, 8, 64):
        _, recv, _, _, _ = run_flat(c5, r)
        assert np.array_equal(recv, brute(c5))
    recv, _, _, _ = run_hier(c5, 8, 8, 8, 8)
    assert np.array_equal(recv, brute(c5))


# ---------------------------------------------------------------- metadata and prefix sums

@pytest.mark.parametrize("P,r", [(8, 2), (9, 3), (16, 4), (13, 2), (20, 5), (12, 12)])
def test_size_tables_follow_the_blocks(P, r):
    """After the rounds of digit x, the block a rank holds for offset o has come
    from the rank (o mod r^(x+1)) places below it; its size is the owner's count."""
    wl = W.make_random(P, 40, elem_size=2, seed=P * r)
    send = wl.make_send().numpy()
    recv = wl.make_recv().numpy().copy()
    _, _, _, _, sizes = oracle.tuna_flat(wl, r, send, recv, want_sizes=True)
    C = wl.sendcounts * wl.elem_size
    for x in range(sizes.shape[0]):
        for p in range(P):
            for o in range(P):
                s = (p - o % r ** (x + 1)) % P
                assert sizes[x, p, o] == C[s, (s + o) % P]


@pytest.mark.parametrize("Q,N,rl,rg", [(5, 3, 2, 3), (4, 4, 2, 2), (3, 4, 3, 2), (6, 5, 2, 3), (8, 4, 8, 4), (1, 5, 2, 2), (5, 1, 2, 2)])
def test_hier_size_tables_follow_the_blocks(Q, N, rl, rg):
    """The metadata the hierarchical schedule holds, by closed form.  After the local
    rounds of digit x the block rank (n, q) holds for rank (i, q + jo) has come from the
    rank (jo mod rl^(x+1)) local places below; the compaction (Sec. IV-B) lists, for every
    group offset, the parts in ascending source local id; after the global rounds of digit
    x a super-block has come (io mod rg^(x+1)) groups; and after the local phase R holds
    the own group's blocks and nothing else (Fig. 5)."""
    P = Q * N
    wl = W.make_random(P, 23, elem_size=3, seed=11 * P + rl + rg, zero_frac=0.25, gaps=True)
    send = wl.make_send().numpy()
    recv = wl.make_recv(fill=CANARY).numpy().copy()
    recv, after, sz_local, usz_compact, usz_global = oracle.tuna_hier_tables(wl, Q, N, rl, rg, send, recv)
    ref = brute(wl)
    assert np.array_equal(recv, ref)
    C = wl.sendcounts * wl.elem_size
    assert sz_local.shape[0] == oracle.num_digits(Q, rl) and usz_global.shape[0] == oracle.num_digits(N, rg)
    for x in range(sz_local.shape[0]):
        for p in range(P):
            n, q = divmod(p, Q)
            for i in range(N):
                for jo in range(Q):
                    qs = (q - jo % rl ** (x + 1)) % Q
                    assert sz_local[x, p, i, jo] == C[n * Q + qs, i * Q + (qs + jo) % Q]
    for p in range(P):
        n, q = divmod(p, Q)
        assert not usz_compact[p, 0].any()                      # the own group's blocks are not compacted
        for io in range(1, N):
            for qs in range(Q):
                assert usz_compact[p, io, qs] == C[n * Q + qs, ((n + io) % N) * Q + q]
    for x in range(usz_global.shape[0]):
        for p in range(P):
            n, q = divmod(p, Q)
            for io in range(1, N):
                n0 = (n - io % rg ** (x + 1)) % N
                for qs in range(Q):
                    assert usz_global[x, p, io, qs] == C[n0 * Q + qs, ((n0 + io) % N) * Q + q]
    own = np.zeros(wl.recv_bytes, dtype=bool)
    for d in range(P):
        for s_ in range(P):
            if s_ // Q == d // Q:
                o = int(wl.recvbase[d] + wl.rdispls[d, s_]) * wl.elem_size
                own[o:o + int(C[s_, d])] = True
    assert np.array_equal(after[own], ref[own]) and np.all(after[~own] == CANARY)


@pytest.mark.parametrize("P,r,threads", [(1, 2, 1), (2, 2, 2), (8, 2, 3), (9, 3, 4), (13, 2, 13), (20, 5, 7), (12, 12, 5),
                                         (33, 6, 8), (64, 64, 16)])
def test_threaded_timing_variant_matches_the_checker(P, r, threads):
    """The threaded variant of the flat schedule exists only to be timed; it must write the
    same bytes (canary gaps included) and count the same rounds as the single-threaded oracle."""
    wl = W.make_random(P, 700, elem_size=3, seed=3 * P + r, zero_frac=0.25, gaps=True)
    send, recv, rounds, _, _ = run_flat(wl, r)
    got = wl.make_recv(fill=CANARY).numpy().copy()
    got, rounds_mt = oracle.tuna_flat_mt(wl, r, send, got, threads)
    assert np.array_equal(got, recv)
    assert np.array_equal(rounds_mt, rounds)


def test_segmented_scan_against_numpy():
    rng = np.random.default_rng(5)
    for nseg, seglen, align in [(1, 1, 1), (3, 7, 1), (5, 33, 16), (64, 64, 16), (2, 100, 4)]:
        v = rng.integers(0, 1000, size=(nseg, seglen)).astype(np.int64)
        v[rng.random(v.shape) < 0.3] = 0
        scan, tot = oracle.segmented_exclusive_scan(v, align)
        pv = (v + align - 1) // align * align
        assert np.array_equal(scan, np.cumsum(pv, axis=1) - pv)
        assert np.array_equal(tot, pv.sum(axis=1))
        assert np.all(scan[:, 0] == 0)
        assert np.array_equal(scan[:, -1] + pv[:, -1], tot)      # last displacement + size = total


# ---------------------------------------------------------------- the paper's other count patterns

def test_paper_count_patterns_small():
    """Normal / power-law sizes (Sec. VI-C) and the two FFT transposes (Sec. VI-A),
    scaled down: shapes as stated in the paper, results equal to the definition."""
    P = 32
    n = W.make_normal(P=P)
    assert n.sendcounts.max() <= 1024 and 850 < n.sendcounts.mean() < 1000    # clipped at the cap
    pl = W.make_powerlaw(P=P)
    assert pl.sendcounts.max() <= 1024 and np.median(pl.sendcounts) < pl.sendcounts.mean()
    f1 = W.make_fft_n1(P=P)
    assert f1.sendcounts.sum() * 1 == math.ceil(0.78125 * P) * math.ceil(0.625 * P) * 8   # = N1
    assert np.all(f1.sendcounts[math.ceil(0.625 * P):] == 0)
    f2 = W.make_fft_n2(P=P)
    assert f2.sendcounts.sum() == ((P - 1) * 32 + 8) * P * 2      # N2 complex values = 2 FP64 each
    for wl in (n, pl, f1, f2):
        ref = brute(wl)
        for r in (2, 8, P):
            _, recv, _, _, _ = run_flat(wl, r)
            assert np.array_equal(recv, ref)
        recv, _, _, _ = run_hier(wl, 8, 4, 8, 4)
        assert np.array_equal(recv, ref)


# ---------------------------------------------------------------- rows with gather / scatter (not in the paper)

def _rows_case(P, maxc, row_bytes, seed, gaps):
    wl = W.make_random(P, maxc, elem_size=row_bytes, seed=seed, zero_frac=0.2, gaps=gaps)
    rng = np.random.default_rng(seed)
    send_rows = wl.send_bytes // row_bytes
    recv_rows = wl.recv_bytes // row_bytes
    in_rows = send_rows + 7
    out_rows = recv_rows + 5
    gather = rng.integers(0, in_rows, send_rows)                 # rows may repeat
    scatter = rng.permutation(out_rows)[:recv_rows]              # injective
    rows_in = rng.integers(0, 256, (in_rows, row_bytes), dtype=np.uint8)
    return wl, gather, scatter, rows_in, out_rows


@pytest.mark.parametrize("P,row_bytes,gaps", [(1, 4, False), (5, 3, True), (8, 16, False), (12, 40, True)])
def test_rows_exchange_is_gather_then_definition_then_scatter(P, row_bytes, gaps):
    wl, gather, scatter, rows_in, out_rows = _rows_case(P, 9, row_bytes, 50 + P, gaps)
    out = np.full((out_rows, row_bytes), CANARY, dtype=np.uint8)
    oracle.rows_alltoallv(wl, gather, scatter, rows_in, out)
    # the same thing from library routines and the pinned definition: numpy take,
    # MPI_Alltoallv on the gathered buffer, numpy fancy assignment
    send = np.ascontiguousarray(rows_in[gather]).reshape(-1)
    recv = oracle.bruteforce(wl, send, np.full(wl.recv_bytes, CANARY, dtype=np.uint8))
    covered = oracle.bruteforce(wl, np.full(wl.send_bytes, 1, dtype=np.uint8),
                                np.zeros(wl.recv_bytes, dtype=np.uint8)).reshape(-1, row_bytes)[:, 0] == 1
    ref = np.full((out_rows, row_bytes), CANARY, dtype=np.uint8)
    ref[scatter[covered]] = recv.reshape(-1, row_bytes)[covered]
    assert np.array_equal(out, ref)
    # identity maps: the plain exchange
    out2 = np.full((wl.recv_bytes // row_bytes, row_bytes), CANARY, dtype=np.uint8)
    rows_send = wl.make_send().numpy().reshape(-1, row_bytes)
    oracle.rows_alltoallv(wl, None, None, rows_send, out2)
    assert np.array_equal(out2.reshape(-1), brute(wl))


def test_rows_exchange_rejects_indices_outside_the_buffers():
    wl, gather, scatter, rows_in, out_rows = _rows_case(4, 5, 8, 3, False)
    out = np.zeros((out_rows, 8), dtype=np.uint8)
    bad = gather.copy()
    bad[0] = rows_in.shape[0]
    if wl.sendcounts[0, 0] == 0:
        bad[:] = rows_in.shape[0]
    with pytest.raises(RuntimeError):
        oracle.rows_alltoallv(wl, bad, scatter, rows_in, out)


def test_moe_row_maps_dispatch_tokens_into_expert_order():
    """Token rows that name their (rank, token): after the exchange every expert holds
    exactly the tokens routed to it, sorted by token index, then by source rank."""
    P, tokens = 8, 64
    wl = W.make_c4(P=P, tokens=tokens, hidden=4)                 # rows of 8 bytes
    first, second = W.moe_top2_routing(wl.seed, P, tokens)
    gather, scatter = W.moe_row_maps(first, second)
    assert np.array_equal(np.bincount(gather, minlength=P * tokens), np.full(P * tokens, 2))
    assert np.array_equal(np.sort(scatter), np.arange(2 * P * tokens))
    rows_in = np.zeros((P * tokens, 8), dtype=np.uint8)
    rows_in[:, 0] = np.repeat(np.arange(P), tokens)
    rows_in[:, 1] = np.tile(np.arange(tokens), P)
    out = np.full((2 * P * tokens, 8), CANARY, dtype=np.uint8)
    oracle.rows_alltoallv(wl, gather, scatter, rows_in, out)
    at = 0
    for d in range(P):
        want = sorted((t, s) for s in range(P) for t in range(tokens)
                      if first[s, t] == d or second[s, t] == d)
        n = len(want)
        assert n == wl.recvcounts[d].sum()
        got = [(int(r[1]), int(r[0])) for r in out[at:at + n]]
        assert got == want
        at += n

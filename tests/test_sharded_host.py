"""Host side of the sharded exchange with two gloo processes on CPU: the rank-to-GPU map,
the all-gather of the count matrix, every GPU's buffer extents and its round table,
against the hierarchical oracle with one group per GPU.  No GPU needed; the data
movement itself is covered by the GPU tests."""
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle
from paper_2411_02581_b200 import binding as B
from paper_2411_02581_b200 import build as build_mod
from paper_2411_02581_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("world", [2, 3])
def test_gloo_processes_agree_with_the_oracle(world):
    build_mod.build()
    import socket
    with socket.socket() as sock:                      # a port that is free right now
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), PYTHONPATH=ROOT,
               CUDA_VISIBLE_DEVICES="")
    procs = [subprocess.Popen([sys.executable, os.path.join(ROOT, "tests", "sharded_worker.py"), str(r),
                               str(world), "cpu"], env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT,
                              text=True) for r in range(world)]
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
        assert p.returncode == 0 and "sharded ok" in outs[r], outs[r]


@pytest.mark.parametrize("P,G,radix", [(8, 2, 2), (12, 3, 0), (16, 4, 4), (15, 5, 2), (6, 6, 2), (7, 1, 3)])
def test_round_table_sums_to_the_oracles_rounds(P, G, radix):
    build_mod.build()
    l = P // G
    wl = W.make_random(P, 90, elem_size=3, seed=P * G, zero_frac=0.3, gaps=True)
    rl = radix if radix else max(2, l)
    _, rounds, _, _ = oracle.tuna_hier(wl, l, G, rl, max(2, G), wl.make_send().numpy(),
                                       wl.make_recv().numpy().copy())
    tables = [B.shard_round_table(P, G, n, radix, wl.elem_size, wl.sendcounts) for n in range(G)]
    for k, row in enumerate(rounds):
        assert all((t[k]["level"], t[k]["x"], t[k]["z"]) == tuple(int(v) for v in row[:3]) for t in tables)
        assert sum(t[k]["bytes"] for t in tables) == row[oracle.RS_BYTES_SENT]
        assert sum(t[k]["units"] for t in tables) == row[oracle.RS_UNITS]
    assert all(len(t) == len(rounds) for t in tables)


def test_layout_rules_and_argument_checks():
    build_mod.build()
    wl = W.make_random(12, 40, elem_size=4, seed=2, zero_frac=0.2, gaps=True)
    G, l, E = 3, 4, 4
    # explicit bases are taken as they are; extents cover the furthest block of each GPU
    sb_in = np.arange(12, dtype=np.int64) % l * 5000
    rb_in = np.arange(12, dtype=np.int64) % l * 7000 + 3
    sb, rb, se, re = B.shard_layout(12, G, E, wl.sendcounts, wl.sdispls, wl.rdispls, sb_in, rb_in)
    assert np.array_equal(sb, sb_in) and np.array_equal(rb, rb_in)
    for n in range(G):
        ranks = range(n * l, (n + 1) * l)
        assert se[n] == max(int(sb_in[p] + (wl.sdispls[p] + wl.sendcounts[p]).max()) for p in ranks) * E
        assert re[n] == max(int(rb_in[p] + (wl.rdispls[p] + wl.sendcounts[:, p]).max()) for p in ranks) * E
    with pytest.raises(B.TunaError, match="BAD_HIERARCHY"):
        B.shard_layout(12, 5, E, wl.sendcounts)
    bad = wl.sendcounts.copy()
    bad[3, 4] = -1
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        B.shard_layout(12, G, E, bad)
    with pytest.raises(B.TunaError, match="INVALID_ARG"):
        B.shard_round_table(12, G, 3, 2, E, wl.sendcounts)
    with pytest.raises(B.TunaError, match="BAD_RADIX"):
        B.shard_round_table(12, G, 0, 5, E, wl.sendcounts)

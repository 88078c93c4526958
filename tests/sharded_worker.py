"""Child process of the sharded tests: one of `world` processes that together run one
sharded exchange.  Usage: sharded_worker.py RANK WORLD [cpu].

With a GPU (every process uses device 0): the whole exchange through ShardedExchange,
checked against the CPU oracle.  With `cpu`: only what needs no GPU (the rank-to-GPU map,
the count all-gather, the layout and the per-GPU round table), checked the same way."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2411_02581_b200 import binding as B  # noqa: E402
from paper_2411_02581_b200 import sharded as S  # noqa: E402
from paper_2411_02581_b200 import workloads as W  # noqa: E402

CANARY = 0xA5


def main():
    rank, world = int(sys.argv[1]), int(sys.argv[2])
    cpu_only = len(sys.argv) > 3 and sys.argv[3] == "cpu"
    dist.init_process_group("gloo", rank=rank, world_size=world)
    P, E, radix = 12 * world, 2, 2
    l = P // world
    wl = W.make_random(P, 600, elem_size=E, seed=77, zero_frac=0.2)          # packed, the same in every process
    mine = S.ranks_of_gpu(P, world, rank)
    assert list(mine) == list(range(rank * l, (rank + 1) * l))
    assert all(S.gpu_of_rank(P, world, p) == rank for p in mine)
    counts = S.gather_counts(wl.sendcounts[mine.start:mine.stop], dist)
    assert np.array_equal(counts, wl.sendcounts)

    send = wl.make_send().numpy()
    ref = wl.make_recv(fill=CANARY).numpy().copy()
    ref, rounds, _, _ = oracle.tuna_hier(wl, l, world, radix, max(2, world), send, ref)
    first = np.arange(world) * l
    cut_s = [int(wl.sendbase[p]) * E for p in first] + [wl.send_bytes]
    cut_r = [int(wl.recvbase[p]) * E for p in first] + [wl.recv_bytes]

    # layout and round table: host only
    sb, rb, se, re = B.shard_layout(P, world, E, counts)
    grp = np.arange(P) // l
    assert np.array_equal(sb, wl.sendbase - wl.sendbase[first][grp])
    assert np.array_equal(rb, wl.recvbase - wl.recvbase[first][grp])
    assert [int(v) for v in se] == [cut_s[n + 1] - cut_s[n] for n in range(world)]
    assert [int(v) for v in re] == [cut_r[n + 1] - cut_r[n] for n in range(world)]
    table = B.shard_round_table(P, world, rank, radix, E, counts)
    assert [(t["level"], t["x"], t["z"]) for t in table] == [tuple(int(v) for v in row[:3]) for row in rounds]
    only = counts.copy()
    only[:rank * l] = 0
    only[(rank + 1) * l:] = 0
    wn = W._finish("shard", P, E, 1, only)
    _, rn, _, _ = oracle.tuna_hier(wn, l, world, radix, max(2, world), wn.make_send().numpy(),
                                   wn.make_recv().numpy().copy())
    assert [t["bytes"] for t in table] == [int(v) for v in rn[:, oracle.RS_BYTES_SENT]]
    # (units count blocks, empty ones included, so every GPU sends its 1/world of them)
    assert [t["units"] * world for t in table] == [int(v) for v in rounds[:, oracle.RS_UNITS]]
    tot = torch.tensor([t["bytes"] for t in table], dtype=torch.int64)
    dist.all_reduce(tot)                                                     # all GPUs together: the oracle's rounds
    assert tot.tolist() == [int(v) for v in rounds[:, oracle.RS_BYTES_SENT]]

    if not cpu_only:
        torch.cuda.set_device(0)
        ex = S.ShardedExchange(P, E, wl.sendcounts[mine.start:mine.stop], radix=radix, dist=dist)
        assert (ex.send_bytes, ex.recv_bytes) == (cut_s[rank + 1] - cut_s[rank], cut_r[rank + 1] - cut_r[rank])
        my_send = torch.from_numpy(send[cut_s[rank]:cut_s[rank + 1]]).cuda()
        d_rows = torch.from_numpy(np.ascontiguousarray(wl.sendcounts[mine.start:mine.stop])).cuda()
        for it in range(3):                                                  # again and again: the buffers are reused
            ex.recv.fill_(CANARY)
            torch.cuda.synchronize()
            if it == 1:
                ex.update_counts(wl.sendcounts[mine.start:mine.stop])        # re-plan from host rows ...
            if it == 2:
                ex.update_counts_device(d_rows)                              # ... and from rows in device memory
            ex.exchange(my_send)
            got = ex.recv[:ex.recv_bytes].cpu().numpy()
            assert np.array_equal(got, ref[cut_r[rank]:cut_r[rank + 1]])
        dist.barrier()
        ex.destroy()
    dist.barrier()
    dist.destroy_process_group()
    print("sharded ok", flush=True)


if __name__ == "__main__":
    main()

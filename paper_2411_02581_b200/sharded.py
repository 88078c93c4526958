"""The exchange with its ranks spread over the GPUs of one node: one process per GPU.

Plumbing only (``torch.distributed`` for the count all-gather, the memory handles
and the closing barrier; torch for device memory): the plan, every copy and the
push into the other GPUs' receive buffers run in the CUDA library
(``tuna_shard_plan_create`` / ``tuna_shard_alltoallv``).

Process ``r`` of the group drives GPU ``r`` and holds the ``l = P / world`` ranks
``r*l .. r*l + l - 1`` (one group of the hierarchical schedule per GPU).
"""
from __future__ import annotations

import numpy as np

from . import binding as B


def ranks_of_gpu(P: int, world: int, gpu: int) -> range:
    """The logical ranks GPU ``gpu`` holds: one group of consecutive ranks."""
    if P % world:
        raise ValueError(f"P = {P} ranks do not divide over {world} GPUs")
    l = P // world
    return range(gpu * l, (gpu + 1) * l)


def gpu_of_rank(P: int, world: int, p: int) -> int:
    return p // (P // world)


def gather_counts(my_rows: np.ndarray, dist=None, group=None) -> np.ndarray:
    """All-gather of the count matrix: every process contributes the rows of its own ranks
    (``[l, P]`` int64, row = sending rank) and gets the full ``[P, P]`` matrix, rows in
    rank order.  Without a process group (one process) the rows are the matrix."""
    import torch
    rows = np.ascontiguousarray(my_rows, dtype=np.int64)
    if dist is None or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return rows.copy()
    world = dist.get_world_size(group)
    backend = dist.get_backend(group)
    dev = torch.device("cuda", torch.cuda.current_device()) if backend == "nccl" else torch.device("cpu")
    mine = torch.from_numpy(rows).to(dev)
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine, group=group)
    return torch.cat(parts, 0).cpu().numpy()


class ShardedExchange:
    """One GPU's share of a sharded exchange, with the buffers and the peers' mappings.

    ``my_rows``: counts ``[l, P]`` of this process's ranks, in elements of ``elem_size``
    bytes.  Layout: every rank's blocks packed in peer order, a GPU's regions packed in
    rank order.  ``recv`` is this GPU's receive buffer (allocated here, exported to the
    other processes); the caller provides the send buffer of ``send_bytes`` bytes.
    """

    def __init__(self, P, elem_size, my_rows, radix=0, dist=None, group=None, device=None):
        import torch
        self.dist, self.group = dist, group
        multi = dist is not None and dist.is_initialized() and dist.get_world_size(group) > 1
        self.world = dist.get_world_size(group) if multi else 1
        self.me = dist.get_rank(group) if multi else 0
        self.P, self.elem_size = P, elem_size
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
        self.counts = gather_counts(my_rows, dist if multi else None, group)
        assert self.counts.shape == (P, P)
        _, _, se, re = B.shard_layout(P, self.world, elem_size, self.counts)
        self.send_bytes, self.recv_bytes = int(se[self.me]), int(re[self.me])
        self.all_recv_bytes = [int(v) for v in re]
        self.plan = B.Plan(P, radix, elem_size=elem_size, sendcounts=self.counts, shard=(self.world, self.me))
        self.workspace = self.plan.alloc_workspace(device=self.device)
        self.recv = torch.empty(max(self.recv_bytes, 16), dtype=torch.uint8, device=self.device)
        self._peers = [None] * self.world      # keeps the mapped tensors alive
        self._peers[self.me] = self.recv
        if multi:
            self._map_peers()
        self._token = torch.zeros(1, dtype=torch.int32, device=self.device)

    def _map_peers(self):
        """Exchange memory handles of the receive buffers and map the others' into this
        process (``torch.multiprocessing``'s CUDA handles); enable peer access for the
        kernels of this GPU."""
        from torch.multiprocessing.reductions import reduce_tensor
        fn, args = reduce_tensor(self.recv)
        handles = [None] * self.world
        self.dist.all_gather_object(handles, (fn, args), group=self.group)
        for r, (f, a) in enumerate(handles):
            if r == self.me:
                continue
            t = f(*a)
            if t.device != self.device:
                rc = B.lib().tuna_shard_enable_peer_access(t.device.index)
                if rc != 0:
                    raise B.TunaError(rc, f"tuna_shard_enable_peer_access({t.device.index})")
            self._peers[r] = t

    def update_counts(self, my_rows):
        """New counts, same shape: all-gather, re-plan, re-size (the receive buffer is kept
        if it is large enough, else it has to be re-created by a new object)."""
        multi = self.world > 1
        self.counts = gather_counts(my_rows, self.dist if multi else None, self.group)
        _, _, se, re = B.shard_layout(self.P, self.world, self.elem_size, self.counts)
        if int(re[self.me]) > self.recv.numel():
            raise ValueError("the receive buffer is too small for the new counts")
        self.send_bytes, self.recv_bytes = int(se[self.me]), int(re[self.me])
        self.plan.update_counts(self.counts)
        if self.plan.workspace_bytes() > self.workspace.numel():
            self.workspace = self.plan.alloc_workspace(device=self.device)

    def update_counts_device(self, my_rows_dev, stream=None):
        """The same from counts in device memory (routing decided on the GPU): ``my_rows_dev``
        is an int64 CUDA tensor ``[l, P]``; the matrix is all-gathered on the device (NCCL;
        with gloo through the host) and the plan re-built from it there.  Only a few totals
        cross back to the host."""
        import torch
        multi = self.world > 1
        if not multi:
            full = my_rows_dev.contiguous()
        elif self.dist.get_backend(self.group) == "nccl":
            full = torch.empty((self.P, self.P), dtype=torch.int64, device=self.device)
            if stream is None:
                self.dist.all_gather_into_tensor(full, my_rows_dev.contiguous(), group=self.group)
            else:
                with torch.cuda.stream(stream):
                    self.dist.all_gather_into_tensor(full, my_rows_dev.contiguous(), group=self.group)
        else:
            full = torch.from_numpy(gather_counts(my_rows_dev.cpu().numpy(), self.dist, self.group)).to(self.device)
        self.plan.update_counts_device(full, stream=stream)
        se, re = self.plan.shard_extents(self.me)
        if re > self.recv.numel():
            raise ValueError("the receive buffer is too small for the new counts")
        self.send_bytes, self.recv_bytes = se, re
        self.counts = None            # (the host copy is stale now)
        if self.plan.workspace_bytes() > self.workspace.numel():
            self.workspace = self.plan.alloc_workspace(device=self.device)

    def _barrier(self, stream):
        import torch
        if self.dist.get_backend(self.group) == "nccl":
            if stream is None:
                self.dist.all_reduce(self._token, group=self.group)
            else:
                with torch.cuda.stream(stream):
                    self.dist.all_reduce(self._token, group=self.group)
        else:
            (torch.cuda.current_stream() if stream is None else stream).synchronize()
            self.dist.barrier(group=self.group)

    def exchange(self, send, stream=None, opening_barrier=True):
        """Enqueue this GPU's share between two barriers across the GPUs.  With NCCL a
        barrier is an all-reduce on the same stream (stream-ordered on every GPU: it
        completes only when every GPU has run what it enqueued before it); otherwise the
        host waits for its own stream and then for the other processes.  The opening
        barrier makes sure every GPU is done with the previous contents of its receive
        buffer before anyone stores into it (skip it if the caller orders that itself);
        the closing one tells every GPU that all stores into its buffer have landed."""
        if self.world > 1 and opening_barrier:
            self._barrier(stream)
        self.plan.shard_alltoallv(send, self._peers, stream=stream)
        if self.world > 1:
            self._barrier(stream)

    def destroy(self):
        self.plan.destroy()
        self._peers = []

"""1D-sharded Dion (Section 4.1, Algorithm 3 of the paper) on top of the library's per-rank calls.

L layers of identical shape m x n are sharded by columns over L ranks (one process per GPU): rank x holds
the columns J_x of every layer's X, M, G and the rows J_x of every layer's right factor.  A step makes three
collectives on flat buffers, whatever L is:

    project all layers locally -> ReduceScatter of the partial panels along L (rank l receives layer l's P)
    -> orthonormalize the owned layer -> AllGather of U (and of the owners' breakdown flags)
    -> W and its squared column norms on the shard -> AllReduce(sum) of r norms per layer -> finish locally.

`torch.distributed` (NCCL over NVLink on GPUs) carries the collectives into this GPU's memory before any
kernel reads the payload; every arithmetic step is in the CUDA library.  The gloo backend of the CPU tests has
no reduce-scatter, so there the partial panels are all-reduced and the owned slice is taken.
"""
from __future__ import annotations

from typing import List, Optional

import torch
import torch.distributed as dist


def _world(group) -> int:
    return dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1


def _rank(group) -> int:
    return dist.get_rank(group) if dist.is_available() and dist.is_initialized() else 0


def reduce_scatter_layers(parts: torch.Tensor, mine: torch.Tensor, group=None) -> None:
    """parts: [L, m, r] partial panels of this rank; mine <- sum over the ranks of parts[rank]."""
    world = _world(group)
    if world == 1:
        mine.copy_(parts[0])
        return
    if parts.is_cuda and dist.get_backend(group) == "nccl":
        dist.reduce_scatter_tensor(mine, parts, op=dist.ReduceOp.SUM, group=group)
    else:
        dist.all_reduce(parts, op=dist.ReduceOp.SUM, group=group)
        mine.copy_(parts[_rank(group)])


def all_gather_layers(allbuf: torch.Tensor, mine: torch.Tensor, group=None) -> None:
    """allbuf: [L, ...]; allbuf[x] <- rank x's `mine`."""
    if _world(group) == 1:
        allbuf[0].copy_(mine.view(allbuf[0].shape))
        return
    if allbuf.is_cuda and dist.get_backend(group) == "nccl":
        dist.all_gather_into_tensor(allbuf, mine, group=group)
    else:       # gloo: one output tensor per rank
        outs = [torch.empty_like(mine) for _ in range(_world(group))]
        dist.all_gather(outs, mine, group=group)
        for x, t in enumerate(outs):
            allbuf[x].copy_(t.view(allbuf[x].shape))


def all_reduce_sum(buf: torch.Tensor, group=None) -> None:
    if _world(group) > 1:
        dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)


class ShardedStepper:
    """Steps L = world-size layers whose column shards this rank holds.

    descs: `binding.DionMatrix` descriptors of this rank's shard of layer 0 .. L-1 (same m, r; n = shard width).
    n_total: the unsharded number of columns."""

    def __init__(self, opt, descs: List, n_total: int, device, group=None):
        self.opt, self.descs, self.group, self.n_total = opt, list(descs), group, int(n_total)
        L = len(self.descs)
        if L != _world(group):
            raise ValueError("1D-sharded Dion steps as many layers as there are ranks")
        m, r, ns = self.descs[0].m, self.descs[0].r, self.descs[0].n
        if any(d.m != m or d.r != r or d.n != ns for d in self.descs):
            raise ValueError("the layers of a sharded step have one shape")
        self.m, self.r = m, r
        self.parts = torch.zeros(L, m, r, dtype=torch.float32, device=device)      # partial P, later U of every layer
        self.mine = torch.zeros(m, r, dtype=torch.float32, device=device)          # the owned layer's P, then U
        self.W = torch.zeros(L, ns, r, dtype=torch.float32, device=device)
        self.sumsq = torch.zeros(L, r, dtype=torch.float32, device=device)
        self.flags = torch.zeros(L, dtype=torch.int32, device=device)
        self.my_flag = torch.zeros(1, dtype=torch.int32, device=device)

    def step(self, lr: float, stream: Optional[torch.cuda.Stream] = None) -> None:
        # the collectives run on torch's current stream: make the caller's stream current for the whole step
        if stream is not None and self.parts.is_cuda:
            with torch.cuda.stream(stream):
                self._step(lr, stream)
        else:
            self._step(lr, stream)

    def _step(self, lr: float, stream) -> None:
        opt, nt = self.opt, self.n_total
        for l, d in enumerate(self.descs):
            opt.shard_project(d, nt, self.parts[l], self.flags[l:l + 1], stream)
        reduce_scatter_layers(self.parts, self.mine, self.group)
        opt.orthonormalize(self.m, self.r, nt, self.mine, self.my_flag, stream)
        all_gather_layers(self.parts, self.mine, self.group)                     # parts[l] <- U of layer l
        all_gather_layers(self.flags, self.my_flag, self.group)                  # flags[l] <- the owner's breakdown flag
        for l, d in enumerate(self.descs):
            opt.shard_factor(d, nt, self.parts[l], self.W[l], self.sumsq[l], self.flags[l:l + 1], stream)
        all_reduce_sum(self.sumsq, self.group)
        for l, d in enumerate(self.descs):
            opt.shard_finish(d, nt, self.parts[l], self.W[l], self.sumsq[l], self.flags[l:l + 1], lr, stream)

"""Compressed data-parallel sync (Section 3.3 of the paper) on top of the three-call C-ABI.

Every data-parallel rank runs one process per GPU with the same X and Q, its own gradient and
its own momentum.  Instead of all-reducing the m x n gradients, the ranks all-reduce the two
low-rank factors of the step: P = (M + G) Q (m x r) and W = (M + G)^T U (n x r).  The factors of
all matrices of a step live in two flat buffers, so a step makes two collectives whatever the
number of matrices.  `torch.distributed` (NCCL over NVLink on GPUs) carries the all-reduce; the
arithmetic of the step is in the CUDA library.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch
import torch.distributed as dist


def all_reduce_mean(buf: torch.Tensor, group=None) -> None:
    """In-place mean over the ranks of `group` (a no-op without an initialised process group).
    On GPUs the division is part of the NCCL collective (ReduceOp.AVG); the gloo backend of the CPU
    tests has no averaging reduction, so there the sum is divided afterwards."""
    if not dist.is_available() or not dist.is_initialized():
        return
    world = dist.get_world_size(group)
    if world == 1:
        return
    if buf.is_cuda and dist.get_backend(group) == "nccl":
        dist.all_reduce(buf, op=dist.ReduceOp.AVG, group=group)
    else:
        dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)
        buf.div_(world)


def flat_views(shapes: Sequence[Sequence[int]], device, dtype=torch.float32, align: int = 4):
    """One flat buffer and a view per shape into it (each view starts on a multiple of `align`
    elements, i.e. 16 bytes for fp32: the library wants 16-byte aligned factors)."""
    offs, total = [], 0
    for shp in shapes:
        offs.append(total)
        n = 1
        for s in shp:
            n *= int(s)
        total += (n + align - 1) // align * align
    flat = torch.zeros(max(total, 1), dtype=dtype, device=device)
    views = []
    for off, shp in zip(offs, shapes):
        n = 1
        for s in shp:
            n *= int(s)
        views.append(flat[off:off + n].view(*shp))
    return flat, views


class DpStepper:
    """Steps a fixed list of matrices with compressed data-parallel sync.

    descs: the `binding.DionMatrix` descriptors of this rank (standard form).  The P, W buffers
    and the per-matrix flags are allocated once."""

    def __init__(self, opt, descs: List, device, group=None):
        self.opt, self.descs, self.group = opt, list(descs), group
        self.flatP, self.P = flat_views([(d.m, d.r) for d in self.descs], device)
        self.flatW, self.W = flat_views([(d.n, d.r) for d in self.descs], device)
        self.flags = torch.zeros(max(len(self.descs), 1), dtype=torch.int32, device=device)

    def step(self, lr: float, stream: Optional[torch.cuda.Stream] = None) -> None:
        """One step.  The library's kernels run on `stream`; the two collectives run on torch's current
        stream, so `stream` is made current for the whole step: otherwise the all-reduces would not be
        ordered against the kernels that write and read the factor buffers."""
        if stream is not None and self.flatP.is_cuda:
            with torch.cuda.stream(stream):
                self._step(lr, stream)
        else:
            self._step(lr, stream)

    def _step(self, lr: float, stream) -> None:
        opt = self.opt
        for k, d in enumerate(self.descs):
            opt.dp_project(d, self.P[k], self.flags[k:k + 1], stream)
        all_reduce_mean(self.flatP, self.group)
        for k, d in enumerate(self.descs):
            opt.dp_factor(d, self.P[k], self.W[k], self.flags[k:k + 1], stream)
        all_reduce_mean(self.flatW, self.group)
        for k, d in enumerate(self.descs):
            opt.dp_finish(d, self.P[k], self.W[k], self.flags[k:k + 1], lr, stream)

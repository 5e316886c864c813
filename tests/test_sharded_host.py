"""Host side of 1D-sharded Dion (Algorithm 3), on CPU: two gloo ranks run the stepper's collectives around a
recording stand-in for the library context; the call order and what each collective delivers are checked."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2504_05295_b200 import sharded


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class _Desc:
    def __init__(self, m, n, r):
        self.m, self.n, self.r = m, n, r


class _RecordingOpt:
    def __init__(self, rank, log):
        self.rank, self.log = rank, log

    def shard_project(self, d, n_total, P, flag, stream=None):
        self.log.append(("project", n_total))
        P.fill_(float(self.rank + 1))                    # every layer's partial panel: 1 on rank 0, 2 on rank 1
        flag.zero_()

    def orthonormalize(self, m, r, n_total, PU, flag, stream=None):
        self.log.append(("orth", float(PU.flatten()[0])))
        PU.fill_(100.0 * (self.rank + 1))                # "U" of the owned layer
        flag.fill_(7 if self.rank == 1 else 0)           # the owner of layer 1 reports a breakdown

    def shard_factor(self, d, n_total, U, W, colsumsq, flag, stream=None):
        self.log.append(("factor", float(U.flatten()[0]), int(flag.item())))
        colsumsq.fill_(float(self.rank + 1))

    def shard_finish(self, d, n_total, U, W, colsumsq, flag, lr, stream=None):
        self.log.append(("finish", float(colsumsq[0]), int(flag.item())))


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    log = []
    stepper = sharded.ShardedStepper(_RecordingOpt(rank, log), [_Desc(6, 4, 3), _Desc(6, 4, 3)], 8, "cpu")
    stepper.step(0.01)
    out[rank] = log
    dist.destroy_process_group()


def test_two_ranks_reduce_scatter_gather_and_reduce():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        logs = [out[r] for r in range(world)]
    for rank, log in enumerate(logs):
        assert [e[0] for e in log] == ["project", "project", "orth", "factor", "factor", "finish", "finish"]
        assert all(e[1] == 8 for e in log if e[0] == "project")           # the unsharded width reaches the library
        # reduce-scatter: the owner of a layer receives the sum of every rank's partial panel, 1 + 2
        assert [e[1] for e in log if e[0] == "orth"] == [3.0]
        # all-gather: every rank sees layer 0's U from rank 0 and layer 1's from rank 1, with the owners' flags
        assert [(e[1], e[2]) for e in log if e[0] == "factor"] == [(100.0, 0), (200.0, 7)]
        # all-reduce of the squared column norms: 1 + 2
        assert [(e[1], e[2]) for e in log if e[0] == "finish"] == [(3.0, 0), (3.0, 7)]


def test_one_rank_needs_no_process_group():
    log = []
    stepper = sharded.ShardedStepper(_RecordingOpt(0, log), [_Desc(5, 3, 2)], 3, "cpu")
    stepper.step(0.01)
    assert [e[0] for e in log] == ["project", "orth", "factor", "finish"]
    assert log[1][1] == 1.0 and log[2][1] == 100.0 and log[3][1] == 1.0


def test_layer_count_must_match_the_ranks():
    import pytest
    with pytest.raises(ValueError):
        sharded.ShardedStepper(_RecordingOpt(0, []), [_Desc(5, 3, 2), _Desc(5, 3, 2)], 3, "cpu")

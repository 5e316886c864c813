"""Host side of the compressed data-parallel sync, on CPU: two gloo ranks average a flat buffer
of low-rank factors, and the call order of a step (project all, all-reduce P, factor all,
all-reduce W, finish all) is checked with a recording stand-in for the library context."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2504_05295_b200 import dp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class _Desc:
    def __init__(self, m, n, r):
        self.m, self.n, self.r = m, n, r


class _RecordingOpt:
    """Stands in for binding.Dion: records the calls and fills the factors with rank-dependent data."""

    def __init__(self, rank, log):
        self.rank, self.log = rank, log

    def dp_project(self, d, P, flag, stream=None):
        self.log.append(("project", d.m))
        P.fill_(float(self.rank + 1))

    def dp_factor(self, d, PU, W, flag, stream=None):
        self.log.append(("factor", d.m, float(PU.flatten()[0])))
        W.fill_(float(10 * (self.rank + 1)))

    def dp_finish(self, d, U, W, flag, lr, stream=None):
        self.log.append(("finish", d.m, float(W.flatten()[0])))


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    log = []
    stepper = dp.DpStepper(_RecordingOpt(rank, log), [_Desc(6, 4, 2), _Desc(3, 5, 1)], "cpu")
    stepper.step(0.01)
    out[rank] = log
    dist.destroy_process_group()


def test_two_ranks_average_both_factors_in_two_collectives():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        logs = [out[r] for r in range(world)]
    for log in logs:
        kinds = [e[0] for e in log]
        assert kinds == ["project", "project", "factor", "factor", "finish", "finish"]
        # ranks wrote 1 and 2 into P, 10 and 20 into W: every rank sees the means 1.5 and 15
        assert all(e[2] == 1.5 for e in log if e[0] == "factor")
        assert all(e[2] == 15.0 for e in log if e[0] == "finish")


def test_flat_views_are_aligned_and_disjoint():
    flat, views = dp.flat_views([(5, 3), (2, 2), (7, 1)], "cpu")
    assert [tuple(v.shape) for v in views] == [(5, 3), (2, 2), (7, 1)]
    starts = [v.data_ptr() - flat.data_ptr() for v in views]
    assert all(s % 16 == 0 for s in starts)
    for k, v in enumerate(views):
        v.fill_(k + 1)
    assert float(views[0].sum()) == 15 and float(views[1].sum()) == 8 and float(views[2].sum()) == 21


def test_all_reduce_mean_without_a_process_group_is_a_no_op():
    t = torch.arange(4.0)
    dp.all_reduce_mean(t)
    assert torch.equal(t, torch.arange(4.0))

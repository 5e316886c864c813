"""1D-sharded Dion (Algorithm 3) through dion_shard_project / dion_orthonormalize / dion_shard_factor /
dion_shard_finish.  The ranks are emulated one after another on the one GPU (each rank's calls run to completion
in stream order; nothing waits on another rank); the three collectives are taken by the test (sum over the
ranks' partial panels, hand-out of U, sum of the squared column norms)."""
import pytest
import torch

from helpers import EPS, ETA, MU, TOL_FP32, rel, to_np64
from oracle import dion_oracle as orc
from paper_2504_05295_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests selected but no CUDA device is visible"
    binding.load_library()


def sharded_step(opt, shards, m, n, r, lr):
    """shards[x][l] = (X, M, G, Q) of rank x's column shard of layer l (device tensors, updated in place)."""
    L = len(shards)
    descs = [[binding.matrix_desc(*shards[x][l]) for l in range(L)] for x in range(L)]
    flag = torch.zeros(L, L, dtype=torch.int32, device="cuda")
    part = [[torch.empty(m, r, device="cuda") for l in range(L)] for x in range(L)]
    for x in range(L):
        for l in range(L):
            opt.shard_project(descs[x][l], n, part[x][l], flag[x, l:l + 1])
    U = []
    oflag = torch.zeros(L, dtype=torch.int32, device="cuda")
    for l in range(L):                                       # rank l owns layer l: reduce-scatter, orthonormalize
        P = torch.stack([part[x][l] for x in range(L)]).sum(0).contiguous()
        opt.orthonormalize(m, r, n, P, oflag[l:l + 1])
        U.append(P)
    W = [[torch.empty(shards[x][l][0].shape[1], r, device="cuda") for l in range(L)] for x in range(L)]
    sq = torch.zeros(L, L, r, device="cuda")
    for x in range(L):                                       # all-gather of U and of the owners' flags
        for l in range(L):
            opt.shard_factor(descs[x][l], n, U[l], W[x][l], sq[x, l], oflag[l:l + 1])
    tot = sq.sum(0).contiguous()                             # all-reduce of the squared column norms
    for x in range(L):
        for l in range(L):
            opt.shard_finish(descs[x][l], n, U[l], W[x][l], tot[l], oflag[l:l + 1], lr)


@pytest.mark.parametrize("ranks,m,n,r", [(2, 512, 768, 128), (3, 384, 600, 96), (4, 1024, 1024, 512), (2, 256, 320, 256)])
def test_sharded_layers_match_the_oracle_and_the_unsharded_step(ranks, m, n, r):
    L = ranks
    pbs = [inputs.make_problem(m, n, r, seed=51, k=l, ks=16) for l in range(L)]
    bounds = orc.shard_bounds(n, L)
    X64 = [to_np64(pb.X) for pb in pbs]; M64 = [to_np64(pb.M) for pb in pbs]; Q64 = [to_np64(pb.Q) for pb in pbs]
    state = [[[pb.X[:, lo:hi].contiguous().cuda(), pb.M[:, lo:hi].contiguous().cuda(), None, pb.Q[lo:hi].contiguous().cuda()]
              for pb in pbs] for (lo, hi) in bounds]
    full_rank = r == min(m, n)
    with binding.Dion(mu=MU, eps=EPS) as opt:
        for t in range(2):
            Gs = [pb.grad(t) for pb in pbs]
            X64, M64, Q64, d64 = orc.sharded_step(X64, M64, [to_np64(g) for g in Gs], Q64, MU, ETA, EPS)
            for x, (lo, hi) in enumerate(bounds):
                for l in range(L):
                    state[x][l][2] = Gs[l][:, lo:hi].contiguous().cuda()
            sharded_step(opt, state, m, n, r, ETA)
        assert opt.get_status() == (0, 0)
    tol = TOL_FP32 if not full_rank else 2e-2      # the full-rank case only checks the plumbing of the adaptive mode
    for l in range(L):
        X = torch.cat([state[x][l][0] for x in range(L)], dim=1)
        M = torch.cat([state[x][l][1] for x in range(L)], dim=1)
        Q = torch.cat([state[x][l][3] for x in range(L)], dim=0)
        ex, em, eq = rel(to_np64(X), X64[l]), rel(to_np64(M), M64[l]), rel(to_np64(Q), Q64[l])
        assert ex <= TOL_FP32 and em <= TOL_FP32 and eq <= tol, (l, ex, em, eq)


def test_one_shard_equals_dion_step_bit_for_bit():
    m, n, r = 768, 512, 128
    pb = inputs.make_problem(m, n, r, seed=52, ks=16, g_dtype=torch.bfloat16)
    G = pb.grad(0).cuda()
    with binding.Dion(mu=MU, eps=EPS) as opt:
        Xa, Ma, Qa = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
        opt.step(Xa, Ma, G, Qa, ETA)
        Xb, Mb, Qb = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
        sharded_step(opt, [[[Xb, Mb, G, Qb]]], m, n, r, ETA)
        assert opt.get_status() == (0, 0)
    assert torch.equal(Xa, Xb) and torch.equal(Ma, Mb) and torch.equal(Qa, Qb)


def test_stepper_with_one_rank():
    from paper_2504_05295_b200 import sharded
    m, n, r = 512, 384, 64
    pb = inputs.make_problem(m, n, r, seed=53, ks=16)
    G = pb.grad(0).cuda()
    with binding.Dion(mu=MU, eps=EPS) as opt:
        Xa, Ma, Qa = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
        opt.step(Xa, Ma, G, Qa, ETA)
        Xb, Mb, Qb = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
        side = torch.cuda.Stream()
        torch.cuda.synchronize()
        sharded.ShardedStepper(opt, [binding.matrix_desc(Xb, Mb, G, Qb)], n, "cuda").step(ETA, side)
        side.synchronize()
        assert opt.get_status(side) == (0, 0)
    assert torch.equal(Xa, Xb) and torch.equal(Ma, Mb) and torch.equal(Qa, Qb)


def test_breakdown_on_the_owner_cancels_the_layer_on_every_shard():
    m, n, r, L = 256, 256, 32, 2
    X = torch.randn(m, n, device="cuda"); M = torch.zeros(m, n, device="cuda")
    G = torch.ones(m, n, device="cuda")                      # rank one: every column of P is the same
    Q = torch.ones(n, r, device="cuda") / n ** 0.5
    h = n // 2
    layer = lambda: [[X[:, :h].clone(), M[:, :h].clone(), G[:, :h].contiguous(), Q[:h].clone()],
                     [X[:, h:].clone(), M[:, h:].clone(), G[:, h:].contiguous(), Q[h:].clone()]]
    a, b = layer(), layer()
    shards = [[a[0], b[0]], [a[1], b[1]]]                    # shards[x][l]
    before = [[t.clone() for t in shards[x][l]] for x in range(L) for l in range(L)]
    with binding.Dion(mu=MU, eps=EPS, orth=binding.ORTH_CHOLQR2) as opt:
        sharded_step(opt, shards, m, n, r, ETA)
        status, skipped = opt.get_status()
    assert status & binding.STATUS_BREAKDOWN and skipped == 4      # two layers x two shards
    after = [shards[x][l] for x in range(L) for l in range(L)]
    for u, v in zip(before, after):
        assert all(torch.equal(p, q) for p, q in zip(u, v))

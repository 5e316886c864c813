"""Compressed data-parallel sync (Section 3.3) through the three-call C-ABI: dion_dp_project,
dion_dp_factor, dion_dp_finish.  The data-parallel ranks are emulated one after another on the
one GPU (each rank's calls run to completion in stream order; nothing waits on another rank), the
all-reduce between the calls is a mean taken by the test."""
import pytest
import torch

from helpers import EPS, ETA, FLOOR_FACTOR, MU, TOL_FP32, one_step_movement, rel, to_np64
from oracle import dion_oracle as orc
from paper_2504_05295_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests selected but no CUDA device is visible"
    binding.load_library()


def dp_step(opt, X_ranks, M_ranks, G_ranks, Q_ranks, d_ranks, lr):
    ranks = len(M_ranks)
    m, n = X_ranks[0].shape
    r = Q_ranks[0].shape[1]
    descs = [binding.matrix_desc(X_ranks[i], M_ranks[i], G_ranks[i], Q_ranks[i], d_ranks[i]) for i in range(ranks)]
    P = [torch.empty(m, r, device="cuda") for _ in range(ranks)]
    W = [torch.empty(n, r, device="cuda") for _ in range(ranks)]
    flag = [torch.zeros(1, dtype=torch.int32, device="cuda") for _ in range(ranks)]
    for i in range(ranks):
        opt.dp_project(descs[i], P[i], flag[i])
    Pm = torch.stack(P).mean(0)                     # the all-reduce (mean) of P
    for i in range(ranks):
        P[i].copy_(Pm)
        opt.dp_factor(descs[i], P[i], W[i], flag[i])
    Wm = torch.stack(W).mean(0)                     # the all-reduce (mean) of W
    for i in range(ranks):
        W[i].copy_(Wm)
        opt.dp_finish(descs[i], P[i], W[i], flag[i], lr)


@pytest.mark.parametrize("m,n,r,ranks", [(256, 512, 64, 2), (640, 384, 96, 3), (1024, 1024, 1024, 2)])
def test_two_and_three_ranks_match_the_oracle(m, n, r, ranks):
    pbs = [inputs.make_problem(m, n, r, seed=31, k=0, ks=16) for _ in range(ranks)]   # same X, Q on every rank
    X64, Q64 = to_np64(pbs[0].X), to_np64(pbs[0].Q)
    M64 = [to_np64(pb.M) for pb in pbs]
    Xs = [pb.X.cuda().clone() for pb in pbs]; Ms = [pb.M.cuda().clone() for pb in pbs]
    Qs = [pb.Q.cuda().clone() for pb in pbs]; ds = [torch.zeros(r, device="cuda") for _ in pbs]
    tol = TOL_FP32
    moved = 0.0
    with binding.Dion(mu=MU, eps=EPS) as opt:
        for t in range(3):
            # rank i sees its own gradient: the seeded gradient of step 3 t + i
            Gs = [pbs[0].grad(3 * t + i) for i in range(ranks)]
            if r == min(m, n):
                # ill-conditioned panel: allow what the float64 rule itself moves by under a float32 panel, summed
                # over the steps (the sync step equals the plain step on the rank-averaged M and G)
                mv = one_step_movement(X64, sum(M64) / ranks, sum(to_np64(g) for g in Gs) / ranks, Q64)
                moved += max(mv.values())
                tol = max(TOL_FP32, FLOOR_FACTOR * moved)
            X64, M64, Q64, d64 = orc.dp_step(X64, M64, [to_np64(g) for g in Gs], Q64, MU, ETA, EPS)
            dp_step(opt, Xs, Ms, [g.cuda() for g in Gs], Qs, ds, ETA)
        assert opt.get_status() == (0, 0)
    for i in range(ranks):
        assert rel(to_np64(Xs[i]), X64) <= tol and rel(to_np64(Qs[i]), Q64) <= tol, i
        assert rel(to_np64(Ms[i]), M64[i]) <= tol, i
        assert torch.equal(Xs[i], Xs[0]) and torch.equal(Qs[i], Qs[0])      # identical weights on every rank
    assert rel(to_np64(ds[0]), d64) <= tol


@pytest.mark.parametrize("precision", [binding.PREC_FP32, binding.PREC_BF16_OPERANDS])
def test_one_rank_equals_dion_step(precision):
    m, n, r = 768, 512, 128
    pb = inputs.make_problem(m, n, r, seed=32, ks=16, g_dtype=torch.bfloat16)
    G = pb.grad(0).cuda()
    with binding.Dion(mu=MU, eps=EPS, precision=precision) as opt:
        Xa, Ma, Qa = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
        opt.step(Xa, Ma, G, Qa, ETA)
        Xb, Mb, Qb = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
        dp_step(opt, [Xb], [Mb], [G], [Qb], [torch.zeros(r, device="cuda")], ETA)
        assert opt.get_status() == (0, 0)
    tol = 0.0 if precision == binding.PREC_FP32 else 2e-2     # bf16 mode: dion_step reads bf16 copies made once
    for name, u, v in (("X", Xa, Xb), ("M", Ma, Mb), ("Q", Qa, Qb)):
        if tol == 0.0:
            assert torch.equal(u, v), name
        else:
            assert rel(to_np64(v), to_np64(u)) <= tol, name


def test_breakdown_in_factor_cancels_finish():
    m, n, r = 256, 256, 32
    X = torch.randn(m, n, device="cuda"); M = torch.zeros(m, n, device="cuda")
    G = torch.ones(m, n, device="cuda")                      # rank one: P has r identical columns
    Q = torch.ones(n, r, device="cuda") / n ** 0.5
    X0, M0, Q0 = X.clone(), M.clone(), Q.clone()
    with binding.Dion(mu=MU, eps=EPS, orth=binding.ORTH_CHOLQR2) as opt:
        dp_step(opt, [X], [M], [G], [Q], [torch.zeros(r, device="cuda")], ETA)
        status, skipped = opt.get_status()
    assert status & binding.STATUS_BREAKDOWN and skipped == 1
    assert torch.equal(X, X0) and torch.equal(M, M0) and torch.equal(Q, Q0)


def test_stepper_with_one_rank_equals_dion_step_on_a_list():
    from paper_2504_05295_b200 import dp
    shapes = [(512, 256, 64), (256, 768, 32), (384, 384, 384)]
    pbs = [inputs.make_problem(m, n, r, seed=33, k=k, ks=16) for k, (m, n, r) in enumerate(shapes)]
    with binding.Dion(mu=MU, eps=EPS) as opt:
        ref = []
        for pb in pbs:
            X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
            opt.step(X, M, pb.grad(0).cuda(), Q, ETA)
            ref.append((X, M, Q))
        got = [(pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()) for pb in pbs]
        Gs = [pb.grad(0).cuda() for pb in pbs]
        descs = [binding.matrix_desc(X, M, G, Q) for (X, M, Q), G in zip(got, Gs)]
        dp.DpStepper(opt, descs, "cuda").step(ETA)
        assert opt.get_status() == (0, 0)
    for k, (a, b) in enumerate(zip(ref, got)):
        for name, u, v in zip("XMQ", a, b):
            assert torch.equal(u, v), f"matrix {k}: {name}"


def test_stepper_on_a_stream_that_is_not_current_orders_its_collectives(monkeypatch):
    # the collectives run on torch's current stream: the stepper must make the caller's stream current,
    # or the all-reduce of P would race the kernels that write and read it
    from paper_2504_05295_b200 import dp
    m, n, r = 1024, 768, 128
    pb = inputs.make_problem(m, n, r, seed=34, ks=16)
    G = pb.grad(0).cuda()
    seen = []

    def fake_all_reduce_mean(buf, group=None):
        seen.append(torch.cuda.current_stream().cuda_stream)
        buf.mul_(1.0)                       # touches the buffer on the current stream, as a collective would

    monkeypatch.setattr(dp, "all_reduce_mean", fake_all_reduce_mean)
    side = torch.cuda.Stream()
    with binding.Dion(mu=MU, eps=EPS) as opt:
        Xa, Ma, Qa = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
        opt.step(Xa, Ma, G, Qa, ETA)
        Xb, Mb, Qb = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
        torch.cuda.synchronize()
        stepper = dp.DpStepper(opt, [binding.matrix_desc(Xb, Mb, G, Qb)], "cuda")
        for _ in range(1):
            stepper.step(ETA, side)
        side.synchronize()
        assert opt.get_status(side) == (0, 0)
    assert seen == [side.cuda_stream, side.cuda_stream]
    assert torch.equal(Xa, Xb) and torch.equal(Ma, Mb) and torch.equal(Qa, Qb)

"""DION_ORTH_RCQR: the randomized Cholesky QR of Algorithm 4 as the step's Orthonormalize,
through the C-ABI, against the float64 oracle that follows the algorithm with the same
sketching matrix (and so, since the result does not depend on the sketch, against the
plain oracle step as well)."""
import pytest
import torch

from helpers import EPS, ETA, MU, TOL_FP32, movement_tol, one_step_movement, oracle_steps, rel, to_np64
from oracle import dion_oracle as orc
from paper_2504_05295_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests selected but no CUDA device is visible"
    binding.load_library()


@pytest.mark.parametrize("engine", [binding.ENGINE_SIMT, binding.ENGINE_AUTO])
@pytest.mark.parametrize("m,n,r,gdt", [(256, 512, 64, torch.float32), (640, 384, 96, torch.float32),
                                       (1536, 1024, 192, torch.bfloat16), (200, 333, 65, torch.float32)])
def test_rcqr_steps_match_the_oracle(engine, m, n, r, gdt):
    pb = inputs.make_problem(m, n, r, seed=27, ks=16, g_dtype=gdt)
    S = inputs.sketch_matrix(pb)
    X64, M64, Q64 = to_np64(pb.X), to_np64(pb.M), to_np64(pb.Q)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
    Sd = S.cuda()
    d = torch.zeros(r, device="cuda")
    with binding.Dion(mu=MU, eps=EPS, orth=binding.ORTH_RCQR, engine=engine) as opt:
        for t in range(4):
            G = pb.grad(t)
            res = orc.step_rcqr(X64, M64, to_np64(G), Q64, to_np64(S), MU, ETA, EPS)
            X64, M64, Q64 = res.X, res.M, res.Q
            opt.step(X, M, G.cuda(), Q, ETA, colnorm_out=d, sketch=Sd)
            if t in (0, 3):
                for name, got, want in (("X", X, res.X), ("M", M, res.M), ("Q", Q, res.Q), ("d", d, res.d)):
                    e = rel(to_np64(got), want)
                    assert e <= TOL_FP32, f"step {t + 1}: {name} off by {e:.2e}"
        assert opt.get_status() == (0, 0)


def test_rcqr_full_rank_panel_and_transposed_form():
    # r = n: the panel B^T Q (n x n) of the transposed form is ill conditioned; one sketch, one Gram matrix
    m, n = 768, 256
    pb = inputs.make_problem(m, n, n, seed=28, ks=16)
    g = torch.Generator(); g.manual_seed(9)
    Q0 = torch.randn(m, n, generator=g); Q0 = Q0 / Q0.norm(dim=0)
    S = inputs.sketch_matrix(pb, transposed=True)
    ref = orc.step_transposed(to_np64(pb.X), to_np64(pb.M), to_np64(pb.grad(0)), to_np64(Q0), MU, ETA, EPS)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), Q0.cuda().clone()
    with binding.Dion(mu=MU, eps=EPS, orth=binding.ORTH_RCQR) as opt:
        opt.step(X, M, pb.grad(0).cuda(), Q, ETA, transposed=True, sketch=S.cuda())
        assert opt.get_status() == (0, 0)
    assert rel(to_np64(M), ref.M) <= TOL_FP32
    # limited by the conditioning of the panel, as in every mode: the conditioned bar of helpers.py
    tol = movement_tol(one_step_movement(to_np64(pb.X), to_np64(pb.M), to_np64(pb.grad(0)), to_np64(Q0), transposed=True))
    ex = rel(to_np64(X), ref.X)
    print(f"rcqr transposed full rank: X {ex:.2e}/{tol['X']:.1e}")
    assert ex <= tol["X"]


def test_rcqr_larger_rank_and_grouped_call():
    shapes = [(2048, 1024, 640), (1024, 2048, 640)]
    pbs = [inputs.make_problem(m, n, r, seed=29, k=k, ks=32) for k, (m, n, r) in enumerate(shapes)]
    Ss = [inputs.sketch_matrix(pb).cuda() for pb in pbs]
    states = [(pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()) for pb in pbs]
    with binding.Dion(mu=MU, eps=EPS, orth=binding.ORTH_RCQR) as opt:
        opt.step_grouped([(X, M, pb.grad(0).cuda(), Q, None, False, S)
                          for pb, (X, M, Q), S in zip(pbs, states, Ss)], ETA)
        assert opt.get_status() == (0, 0)
    for pb, (X, M, Q) in zip(pbs, states):
        ref = oracle_steps(pb, 1)[0]
        assert rel(to_np64(X), ref.X) <= TOL_FP32 and rel(to_np64(M), ref.M) <= TOL_FP32
        assert rel(to_np64(Q), ref.Q) <= TOL_FP32


def test_rcqr_needs_a_sketch():
    pb = inputs.make_problem(256, 128, 32, seed=30, ks=8)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
    with binding.Dion(orth=binding.ORTH_RCQR) as opt:
        with pytest.raises(binding.DionError):
            opt.step(X, M, pb.grad(0).cuda(), Q, ETA)
        with pytest.raises(binding.DionError):          # too few rows
            opt.step(X, M, pb.grad(0).cuda(), Q, ETA, sketch=torch.randn(16, 256, device="cuda"))
        assert opt.get_status() == (0, 0)
    assert torch.equal(X, pb.X.cuda())

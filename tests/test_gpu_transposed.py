"""The transposed form of the Dion step (Section 4.3, "other variants": the power
iteration runs on M^T) through the C-ABI, against the float64 oracle's
`step_transposed` (= the standard step on the transposed arrays).

The warm-start factor Q lives on the row side (m x r) and the orthonormalized panel
on the column side (n x r), which is the cheaper side when m > n.
"""
import numpy as np
import pytest
import torch

from helpers import EPS, ETA, MU, TOL_BF16, TOL_FP32, movement_tol, one_step_movement, rel, to_np64
from oracle import dion_oracle as orc
from paper_2504_05295_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests selected but no CUDA device is visible"
    binding.load_library()


def row_side_factor(m, r, seed):
    g = torch.Generator(); g.manual_seed(seed)
    Q = torch.randn(m, r, generator=g)
    return Q / Q.norm(dim=0)


def oracle_chain(pb, Q0, steps):
    X, M, Q = to_np64(pb.X), to_np64(pb.M), to_np64(Q0)
    out = []
    for t in range(steps):
        res = orc.step_transposed(X, M, to_np64(pb.grad(t)), Q, MU, ETA, EPS)
        X, M, Q = res.X, res.M, res.Q
        out.append(res)
    return out


@pytest.mark.parametrize("engine", [binding.ENGINE_SIMT, binding.ENGINE_AUTO])
@pytest.mark.parametrize("m,n,r,gdt", [(640, 384, 96, torch.float32), (384, 640, 96, torch.float32),
                                       (257, 129, 33, torch.float32), (1792, 512, 128, torch.bfloat16),
                                       (512, 1792, 128, torch.bfloat16), (2048, 1024, 256, torch.float32)])
def test_transposed_form_matches_oracle(engine, m, n, r, gdt):
    pb = inputs.make_problem(m, n, r, seed=23, ks=16, g_dtype=gdt)
    Q0 = row_side_factor(m, r, 5)
    ref = oracle_chain(pb, Q0, 3)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), Q0.cuda().clone()
    d = torch.zeros(r, device="cuda")
    with binding.Dion(mu=MU, eps=EPS, engine=engine) as opt:
        for t in range(3):
            opt.step(X, M, pb.grad(t).cuda(), Q, ETA, colnorm_out=d, transposed=True)
            if t in (0, 2):
                for name, got, want in (("X", X, ref[t].X), ("M", M, ref[t].M), ("Q", Q, ref[t].Q), ("d", d, ref[t].d)):
                    e = rel(to_np64(got), want)
                    assert e <= TOL_FP32, f"step {t + 1}: {name} off by {e:.2e}"
        assert opt.get_status() == (0, 0)


def test_transposed_full_rank_on_the_short_side():
    # r = n < m: the n x n panel is square and ill conditioned -> adaptive rounds; M' = mu B exactly
    m, n = 1536, 512
    pb = inputs.make_problem(m, n, n, seed=24, ks=16)
    Q0 = row_side_factor(m, n, 6)
    ref = oracle_chain(pb, Q0, 1)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), Q0.cuda().clone()
    B = to_np64(M) + to_np64(pb.grad(0))
    with binding.Dion(mu=MU, eps=EPS) as opt:
        opt.step(X, M, pb.grad(0).cuda(), Q, ETA, transposed=True)
        assert opt.get_status() == (0, 0)
    assert rel(to_np64(M), MU * B) <= TOL_FP32
    assert rel(to_np64(M), ref[0].M) <= TOL_FP32
    # the update itself is only as well determined as the panel's conditioning allows: 1e-4, or what the
    # float64 rule moves by under a float32 panel on this input (helpers.py)
    tol = movement_tol(one_step_movement(to_np64(pb.X), to_np64(pb.M), to_np64(pb.grad(0)), to_np64(Q0), transposed=True))
    ex, eq = rel(to_np64(X), ref[0].X), rel(to_np64(Q), ref[0].Q)
    print(f"transposed full rank: X {ex:.2e}/{tol['X']:.1e} Q {eq:.2e}/{tol['Q']:.1e}")
    assert ex <= tol["X"] and eq <= tol["Q"]


def test_grouped_list_mixes_both_forms():
    m, n, r = 768, 256, 64
    pbs = [inputs.make_problem(m, n, r, seed=25, k=k, ks=16) for k in range(4)]
    forms = [False, True, True, False]
    Q0 = [pb.Q if not tr else row_side_factor(m, r, 30 + k) for k, (pb, tr) in enumerate(zip(pbs, forms))]
    single = []
    with binding.Dion(mu=MU, eps=EPS) as opt:
        for pb, q, tr in zip(pbs, Q0, forms):
            X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), q.cuda().clone()
            opt.step(X, M, pb.grad(0).cuda(), Q, ETA, transposed=tr)
            single.append((X, M, Q))
        grouped = [(pb.X.cuda().clone(), pb.M.cuda().clone(), q.cuda().clone()) for pb, q in zip(pbs, Q0)]
        opt.step_grouped([(X, M, pb.grad(0).cuda(), Q, None, tr)
                          for pb, (X, M, Q), tr in zip(pbs, grouped, forms)], ETA)
        assert opt.get_status() == (0, 0)
    for k, (a, b) in enumerate(zip(single, grouped)):
        for name, u, v in zip("XMQ", a, b):
            assert torch.equal(u, v), f"matrix {k}: {name} differs between dion_step and dion_step_grouped"
    for pb, q, tr, (X, M, Q) in zip(pbs, Q0, forms, grouped):
        f = orc.step_transposed if tr else orc.step
        res = f(to_np64(pb.X), to_np64(pb.M), to_np64(pb.grad(0)), to_np64(q), MU, ETA, EPS)
        assert rel(to_np64(X), res.X) <= TOL_FP32 and rel(to_np64(M), res.M) <= TOL_FP32
        assert rel(to_np64(Q), res.Q) <= TOL_FP32


def test_transposed_argument_checks():
    m, n, r = 256, 128, 32
    X = torch.zeros(m, n, device="cuda"); M = torch.zeros(m, n, device="cuda")
    G = torch.ones(m, n, device="cuda"); Qm = torch.ones(m, r, device="cuda")
    with binding.Dion() as opt:
        with pytest.raises(ValueError):
            opt.step(X, M, G, Qm, ETA)                          # m x r factor without the flag
        with pytest.raises(binding.DionError):
            d = binding.matrix_desc(X, M, G, Qm, None, True)
            d.transposed = 2
            opt.step_desc(d, ETA, int(torch.cuda.current_stream().cuda_stream))
        with pytest.raises(binding.DionError):                  # Algorithm 6 exists in the standard form only
            d = binding.matrix_desc(X, M, G, Qm, None, True)
            binding._check(opt._lib.dion_lazy_step(opt._ctx, d, ETA, 1, int(torch.cuda.current_stream().cuda_stream)))
        assert opt.get_status() == (0, 0)


@pytest.mark.parametrize("m,n,r", [(1024, 512, 128), (520, 1032, 72), (1000, 776, 100)])
def test_transposed_form_in_bf16_operand_mode(m, n, r):
    # the first two shapes take the bf16-array products (every dimension a multiple of 8), the last one
    # the variant that rounds fp32 tiles inside the kernel
    pb = inputs.make_problem(m, n, r, seed=26, ks=16, g_dtype=torch.bfloat16)
    Q0 = row_side_factor(m, r, 7)
    ref = oracle_chain(pb, Q0, 5)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), Q0.cuda().clone()
    with binding.Dion(mu=MU, eps=EPS, precision=binding.PREC_BF16_OPERANDS) as opt:
        for t in range(5):
            opt.step(X, M, pb.grad(t).cuda(), Q, ETA, transposed=True)
        assert opt.get_status() == (0, 0)
    for name, got, want in (("X", X, ref[4].X), ("M", M, ref[4].M), ("Q", Q, ref[4].Q)):
        e = rel(to_np64(got), want)
        assert e <= TOL_BF16, f"{name} off by {e:.2e}"


def test_transposed_form_at_a_llama_shape_with_bf16_gradients():
    # 14336 x 4096 at r = 1024 in the transposed form (the panel on the 4096 side): large enough for P on bf16 pairs
    # with the probe-gated recomputation, the Gram matrix on half pairs and the chain of 512-column blocks
    m, n, r = 14336, 4096, 1024
    pb = inputs.make_problem(m, n, r, seed=29, ks=64, g_dtype=torch.bfloat16)
    Q0 = row_side_factor(m, r, 7)
    want = orc.step_transposed(to_np64(pb.X), to_np64(pb.M), to_np64(pb.grad(0)), to_np64(Q0), MU, ETA, EPS)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), Q0.cuda().clone()
    d = torch.zeros(r, device="cuda")
    with binding.Dion(mu=MU, eps=EPS) as opt:
        opt.step(X, M, pb.grad(0).cuda(), Q, ETA, colnorm_out=d, transposed=True)
        assert opt.get_status() == (0, 0) and opt.orth_rounds() == 1
    errs = {"X": rel(to_np64(X), want.X), "M": rel(to_np64(M), want.M), "Q": rel(to_np64(Q), want.Q), "d": rel(to_np64(d), want.d)}
    print("transposed 14336 x 4096 r=1024: " + " ".join(f"{k} {v:.2e}" for k, v in errs.items()))
    assert all(v <= TOL_FP32 for v in errs.values()), errs

"""Parity at the sizes the benchmark times (needs a B200; ``-m gpu``).

Three layers:
* element-by-element comparison with the float64 oracle at the full-rank squares the oracle still
  finishes in minutes (2048^2 after 1 and 10 steps, 4096^2 after 1 step), in the default (AUTO) mode;
* a pin of the orthonormal basis that holds at any size: with P0 = (M + G) Q and U as the library
  computes them (the data-parallel entry points hand both out), T = U^T P0 must be upper triangular
  with a positive diagonal and U T = P0, i.e. U is the thin-QR factor of P0 and not merely some
  orthonormal basis; evaluated in float64 on the device by the test;
* a row-sampled oracle comparison for a matrix too large for the full oracle step.
"""
import numpy as np
import pytest
import torch

from helpers import (EPS, ETA, MU, TOL_FP32, check_conditioned, oracle_steps, oracle_steps_fp32_panel, rel,
                     to_np64)
from oracle import dion_oracle as orc
from paper_2504_05295_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests selected but no CUDA device is visible"
    binding.load_library()


def _state(X, M, Q, d):
    return (to_np64(X), to_np64(M), to_np64(Q), to_np64(d))


def test_2048_square_full_rank_auto_after_1_and_10_steps():
    # cond(P) is 1e5 .. 1e7 here: the bar is the conditioned one of helpers.py (1e-4 wherever the float64
    # rule itself is that well determined)
    n = 2048
    pb = inputs.make_problem(n, n, n, seed=21, ks=64)
    ref = oracle_steps(pb, 10)
    moved = oracle_steps_fp32_panel(pb, 10)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
    d = torch.zeros(n, device="cuda")
    with binding.Dion(mu=MU, eps=EPS) as opt:               # AUTO: the adaptive Cholesky-QR rounds
        for t in range(10):
            opt.step(X, M, pb.grad(t).cuda(), Q, ETA, colnorm_out=d)
            if t == 0:
                first = _state(X, M, Q, d)
        assert opt.get_status() == (0, 0)
    check_conditioned(first, ref[0], moved[0], "2048^2 full rank, step 1")
    errs, _ = check_conditioned(_state(X, M, Q, d), ref[9], moved[9], "2048^2 full rank, step 10")
    assert errs["M"] <= TOL_FP32          # M_new = mu (M + G) at full rank whatever U is


def test_4096_square_full_rank_auto_step_1():
    n = 4096
    pb = inputs.make_problem(n, n, n, seed=22, ks=64)
    ref = oracle_steps(pb, 1)
    moved = oracle_steps_fp32_panel(pb, 1)
    X, M, Q = pb.X.cuda().clone(), pb.M.cuda().clone(), pb.Q.cuda().clone()
    d = torch.zeros(n, device="cuda")
    with binding.Dion(mu=MU, eps=EPS) as opt:
        opt.step(X, M, pb.grad(0).cuda(), Q, ETA, colnorm_out=d)
        assert opt.get_status() == (0, 0)
    errs, _ = check_conditioned(_state(X, M, Q, d), ref[0], moved[0], "4096^2 full rank, step 1")
    assert errs["X"] <= TOL_FP32 and errs["M"] <= TOL_FP32


def basis_pin(m, n, r, g_dtype, warm_steps=1):
    """P0 and U of the step that follows `warm_steps` ordinary steps, checked in float64."""
    pb = inputs.make_problem(m, n, r, seed=23, ks=64, g_dtype=g_dtype, device="cuda", keep_signal=False)
    X, M, Q = pb.X, pb.M, pb.Q
    P = torch.empty(m, r, device="cuda")
    W = torch.empty(n, r, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    with binding.Dion(mu=MU, eps=EPS) as opt:
        for t in range(warm_steps):
            opt.step(X, M, pb.grad(t), Q, ETA)
        G = pb.grad(warm_steps)
        desc = binding.matrix_desc(X, M, G, Q)
        opt.dp_project(desc, P, flag)
        P0 = P.double()
        opt.dp_factor(desc, P, W, flag)                     # P <- U, W <- (M + G)^T U
        assert opt.get_status() == (0, 0) and int(flag.item()) == 0
        U = P.double()
        # the step itself, from the same state: its update must be built from this U
        X0 = X.clone()
        d = torch.zeros(r, device="cuda")
        opt.step(X, M, G, Q, ETA, colnorm_out=d)
        assert opt.get_status() == (0, 0)
    del P
    # P0 = (M0 + G) Q_old on sampled rows (float64 product of the same fp32 / bf16 inputs): the state
    # before the last step is gone, so this is checked through U T = P0 and W below instead
    T = U.t() @ P0
    nT = float(torch.linalg.norm(T))
    low = float(torch.linalg.norm(torch.tril(T, -1))) / nT
    diag_min = float(torch.diagonal(T).min())
    recon = float(torch.linalg.norm(U @ T - P0) / torch.linalg.norm(P0))
    del T
    eye_dev = float((U.t() @ U - torch.eye(r, device="cuda", dtype=torch.float64)).abs().max())
    # the step's own update: (X0 - X') / s = U Q'^T with the Q' it wrote
    s = ETA * (m / n) ** 0.5
    upd = (X0.double() - X.double()) / s
    upd_err = float(torch.linalg.norm(upd - U @ Q.double().t()) / torch.linalg.norm(upd))
    # W = (M + G)^T U (its column norms are the exported d)
    d_err = float(torch.linalg.norm(torch.linalg.norm(W.double(), dim=0) - d.double()) / torch.linalg.norm(d.double()))
    print(f"{m}x{n} r={r}: tril {low:.2e} diag_min {diag_min:.3e} recon {recon:.2e} orth {eye_dev:.2e} "
          f"update {upd_err:.2e} d {d_err:.2e}")
    assert low <= TOL_FP32 and diag_min > 0.0 and recon <= TOL_FP32
    assert eye_dev <= TOL_FP32
    # the update product runs single-pass TF32 on factors rounded to nearest (relative operand error <= 2^-11,
    # unbiased: ~3e-4 on the update, ~3e-6 on X), and X is fp32: the eta-scaled update is read back by subtraction
    assert upd_err <= 1e-3
    assert d_err <= TOL_FP32
    torch.cuda.empty_cache()


@pytest.mark.parametrize("m,n,r", [(2048, 2048, 2048), (4096, 4096, 4096), (8192, 8192, 8192), (8192, 8192, 2048)])
def test_thin_qr_basis_on_the_square_sweep(m, n, r):
    basis_pin(m, n, r, torch.float32)


@pytest.mark.parametrize("m,n,r", [(16384, 16384, 4096), (16384, 16384, 256), (32768, 32768, 2048)])
def test_thin_qr_basis_on_the_large_squares(m, n, r):
    basis_pin(m, n, r, torch.float32, warm_steps=0 if m > 16384 else 1)


@pytest.mark.parametrize("m,n,r", [(14336, 4096, 1024), (4096, 14336, 1024), (53248, 16384, 1024), (16384, 53248, 1024)])
def test_thin_qr_basis_on_llama_shapes_bf16_gradients(m, n, r):
    basis_pin(m, n, r, torch.bfloat16, warm_steps=0 if max(m, n) > 16384 else 1)


def test_16384_square_r1024_against_row_sampled_oracle():
    # the oracle's factors for the whole matrix (P0, Householder QR of the 16384 x 1024 panel, W, ColNorm),
    # its M_new and X_new on 256 random rows; Q_new and d in full
    m = n = 16384
    r = 1024
    pb = inputs.make_problem(m, n, r, seed=24, ks=64)
    G = pb.grad(0)
    rows = np.sort(np.random.default_rng(24).choice(m, size=256, replace=False))
    Xr, Mr, Qn, dn = orc.step_rows(to_np64(pb.X), to_np64(pb.M), to_np64(G), to_np64(pb.Q), rows, MU, ETA, EPS)
    X, M, Q = pb.X.cuda(), pb.M.cuda(), pb.Q.cuda()
    d = torch.zeros(r, device="cuda")
    with binding.Dion(mu=MU, eps=EPS) as opt:
        opt.step(X, M, G.cuda(), Q, ETA, colnorm_out=d)
        assert opt.get_status() == (0, 0)
    idx = torch.from_numpy(rows).cuda()
    errs = {"X rows": rel(to_np64(X[idx]), Xr), "M rows": rel(to_np64(M[idx]), Mr),
            "Q": rel(to_np64(Q), Qn), "d": rel(to_np64(d), dn)}
    # the update itself on those rows (X alone would hide it behind |X| >> |update|)
    upd_g = to_np64(pb.X[rows]) - to_np64(X[idx])
    upd_o = to_np64(pb.X[rows]) - Xr
    errs["update rows"] = rel(upd_g, upd_o)
    print("16384^2 r=1024: " + " ".join(f"{k} {v:.2e}" for k, v in errs.items()))
    assert errs["X rows"] <= TOL_FP32 and errs["M rows"] <= TOL_FP32 and errs["Q"] <= TOL_FP32 and errs["d"] <= TOL_FP32
    # the update: single-pass TF32 on rounded factors (~3e-4), read back by subtraction from fp32 X
    assert errs["update rows"] <= 1e-3
    torch.cuda.empty_cache()

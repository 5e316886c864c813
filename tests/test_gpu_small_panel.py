"""CholeskyQR2 of a panel that fits one CTA's shared memory (r <= 64, at most 512 rows: one launch) through
dion_orthonormalize, against what fixes the thin-QR factor (Section 3.2 of the paper: Orthonormalize returns the
orthonormal factor of a QR decomposition): U^T U = I, U T = P with T upper triangular and a positive diagonal.
Computed in float64 by the test from the kernel's U and the input panel."""
import numpy as np
import pytest
import torch

from paper_2504_05295_b200 import binding, build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests selected but no CUDA device is visible"
    binding.load_library()


def panel(rows, r, cond, seed):
    """rows x r with singular values log-spaced from 1 to 1 / cond (orthonormal factors from seeded Gaussians)."""
    rng = np.random.default_rng(seed)
    A, _ = np.linalg.qr(rng.standard_normal((rows, r)))
    B, _ = np.linalg.qr(rng.standard_normal((r, r)))
    s = np.logspace(0.0, -np.log10(cond), r) if r > 1 else np.ones(1)
    return (A * s) @ B.T


def check_factor(U, P, tol_orth, tol_fit):
    r = P.shape[1]
    E = U.T @ U - np.eye(r)
    assert np.abs(E).max() <= tol_orth, np.abs(E).max()
    T = U.T @ P
    assert np.all(np.diag(T) > 0)
    assert np.linalg.norm(np.tril(T, -1)) <= tol_fit * np.linalg.norm(T)
    assert np.linalg.norm(U @ T - P) <= tol_fit * np.linalg.norm(P)


# 513 rows and r = 65 take the launch chain of the larger panels: same checks on both sides of the size rule
@pytest.mark.parametrize("rows,r", [(256, 64), (512, 64), (130, 10), (100, 37), (64, 64), (77, 1), (300, 48), (513, 64), (256, 65)])
@pytest.mark.parametrize("cond", [3.0, 300.0])
def test_small_panel_factor_is_the_thin_qr_factor(rows, r, cond):
    P = panel(rows, r, cond, seed=rows + r)
    with binding.Dion(mu=0.95, eps=1e-8, orth=binding.ORTH_CHOLQR2) as opt:
        PU = torch.from_numpy(P).float().cuda().contiguous()
        P32 = PU.double().cpu().numpy()              # what the kernel was given
        flag = torch.zeros(1, dtype=torch.int32, device="cuda")
        opt.orthonormalize(rows, r, 8 * max(r, 8), PU, flag)
        rounds = opt.orth_rounds()
        assert opt.get_status() == (0, 0) and int(flag.item()) == 0
    U = PU.double().cpu().numpy()
    # cond 3: one round is orthonormal to the test's threshold; cond 300: the first round leaves ~cond^2 eps and the
    # second runs (on the small panels: inside the same launch)
    assert rounds == (1 if (cond < 10 or r == 1) else 2), rounds      # (a single column has condition number 1)
    check_factor(U, P32, 2e-5, 2e-5 if cond < 10 else 2e-4)


def test_small_panel_in_a_grouped_chain_equals_single_calls_and_is_reproducible():
    from helpers import EPS, ETA, MU, device_state
    from paper_2504_05295_b200 import inputs
    pbs = [inputs.make_problem(256, 512, 64, seed=3, k=k, ks=16) for k in range(5)]
    runs = []
    for rep in range(2):
        with binding.Dion(mu=MU, eps=EPS) as opt:
            states = [device_state(pb) for pb in pbs]
            for t in range(3):
                opt.step_grouped([(X, M, pb.grad(t).cuda(), Q) for pb, (X, M, Q) in zip(pbs, states)], ETA)
            assert opt.get_status() == (0, 0)
        runs.append(states)
    with binding.Dion(mu=MU, eps=EPS) as opt:
        single = [device_state(pb) for pb in pbs]
        for pb, (X, M, Q) in zip(pbs, single):
            for t in range(3):
                opt.step(X, M, pb.grad(t).cuda(), Q, ETA)
    for a, b, c in zip(runs[0], runs[1], single):
        for u, v, w in zip(a, b, c):
            assert torch.equal(u, v) and torch.equal(u, w)

"""Pins of the float64 CPU oracle against what the paper and the mathematics fix.

None of these tests needs a GPU.  Each pin is chosen so that a plausible
mistake in the oracle (a dropped term, a wrong sign or index, a transposed
operand, the wrong operand in ColNorm or in the error feedback) fails at least
one of them.  Library routines (numpy QR / SVD) are used only as independent
references; the oracle itself never calls them.
"""
import os

import numpy as np
import pytest

from oracle import dion_oracle as orc

MU, ETA, EPS = 0.95, 0.01, 1e-8
HERE = os.path.dirname(os.path.abspath(__file__))


def rel(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def orth(rng, rows, cols):
    q, rr = np.linalg.qr(rng.standard_normal((rows, cols)))
    return q * np.sign(np.diag(rr))


def draw(rng, m, n, r):
    X = 0.02 * rng.standard_normal((m, n))
    M = rng.standard_normal((m, n))
    G = rng.standard_normal((m, n))
    Q = rng.standard_normal((n, r))
    Q /= np.linalg.norm(Q, axis=0)
    return X, M, G, Q


def load_golden(name):
    out = {}
    with open(os.path.join(HERE, "golden", name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            tok = line.split()
            rows, cols = int(tok[1]), int(tok[2])
            out[tok[0]] = np.array([float(t) for t in tok[3:]]).reshape(rows, cols)
    return out


# -- hand-worked fixture (Algorithm 1 + 2 by pencil) --------------------------

def test_hand_worked_2x2_fixture():
    g = load_golden("hand_2x2.txt")
    M = np.array([[1.0, 0.0], [1.0, 1.0]])
    G = np.array([[2.0, 1.0], [3.0, 1.0]])
    res = orc.step(np.zeros((2, 2)), M, G, np.eye(2), mu=0.95, eta=0.1, eps=0.0)
    assert np.allclose(res.U, g["U"], atol=1e-14)
    assert np.allclose(res.R, g["W"], atol=1e-14)
    assert np.allclose(res.M, g["M_new"], atol=1e-14)
    assert np.allclose(res.d, g["d"].ravel(), atol=1e-14)
    assert np.allclose(res.Q, g["V_new"], atol=1e-14)
    assert np.allclose(res.X, g["X_new"], atol=1e-14)


# -- pin 1 / 10: orthonormal factor, cross-check with a library QR ------------

@pytest.mark.parametrize("m,r", [(7, 1), (9, 9), (40, 6), (257, 33)])
def test_householder_matches_library_qr(m, r):
    rng = np.random.default_rng(10 + m + r)
    P = rng.standard_normal((m, r)) * np.logspace(0, -3, r)
    U, Rq = orc.householder_qr(P)
    q, rr = np.linalg.qr(P)
    s = np.sign(np.diag(rr))
    assert np.abs(U.T @ U - np.eye(r)).max() < 1e-13 * r
    assert np.all(np.diag(Rq) > 0)
    assert np.allclose(np.tril(Rq, -1), 0)
    assert rel(U @ Rq, P) < 1e-13
    assert rel(U, q * s) < 1e-11
    assert rel(Rq, (rr.T * s).T) < 1e-11


def test_householder_negative_leading_entries_and_zero_column():
    # leading entries of both signs exercise the alpha sign choice and the sign fix
    P = np.array([[-3.0, 1.0], [4.0, -2.0], [0.0, 5.0]])
    U, Rq = orc.householder_qr(P)
    assert np.all(np.diag(Rq) > 0) and rel(U @ Rq, P) < 1e-14
    assert np.allclose(U[:, 0], [-0.6, 0.8, 0.0], atol=1e-14)
    # an all-zero column: identity reflector, finite output
    Pz = np.zeros((5, 2)); Pz[:, 1] = [1, 2, 3, 4, 5]
    Uz, Rz = orc.householder_qr(Pz)
    assert np.all(np.isfinite(Uz)) and np.abs(Uz.T @ Uz - np.eye(2)).max() < 1e-13


# -- pin 2: ColNorm ------------------------------------------------------------

def test_colnorm_definition_and_zero_column():
    rng = np.random.default_rng(2)
    W = rng.standard_normal((13, 4)); W[:, 2] = 0.0
    Wn, d = orc.colnorm(W, 1e-8)
    ref = np.sqrt((W * W).sum(0))
    assert np.allclose(d, ref, rtol=1e-15)
    assert np.all(Wn[:, 2] == 0.0) and np.all(np.isfinite(Wn))
    nz = [0, 1, 3]
    assert np.allclose(np.linalg.norm(Wn[:, nz], axis=0), ref[nz] / (ref[nz] + 1e-8), rtol=1e-14)
    assert np.allclose(Wn[:, nz] * (ref[nz] + 1e-8), W[:, nz], rtol=1e-14)


# -- pin 1, 3: invariants of one step -----------------------------------------

@pytest.mark.parametrize("m,n,r", [(24, 40, 6), (40, 24, 6), (33, 33, 33), (64, 48, 1)])
def test_step_invariants(m, n, r):
    rng = np.random.default_rng(100 + m + n + r)
    X, M, G, Q = draw(rng, m, n, r)
    res = orc.step(X, M, G, Q, MU, ETA, EPS)
    B = M + G
    U, R = res.U, res.R
    assert res.degenerate == 0
    assert rel(res.P, B @ Q) < 1e-14                       # P = B V (not B^T, not M alone)
    assert np.abs(U.T @ U - np.eye(r)).max() < 1e-13 * r   # U orthonormal
    assert rel(U @ (U.T @ res.P), res.P) < 1e-13           # range(U) = range(P)
    assert rel(R, B.T @ U) < 1e-14                         # W = B^T U
    # error feedback, Eq. 1: M_new = (1-beta) B + beta (B - U W^T) = B - beta U W^T
    assert rel(res.M + (1 - MU) * U @ R.T, B) < 1e-13
    assert rel(U.T @ res.M, MU * (U.T @ B)) < 1e-12        # projector form
    comp = (res.M - U @ (U.T @ res.M)) - (B - U @ (U.T @ B))     # untouched complement
    assert np.linalg.norm(comp) < 1e-12 * np.linalg.norm(B)
    # ColNorm uses the un-normalised W and feeds the update
    assert np.allclose(res.d, np.linalg.norm(R, axis=0), rtol=1e-14)
    assert rel(res.Q, R / (res.d + EPS)) < 1e-14
    assert rel(res.X, X - ETA * np.sqrt(m / n) * U @ res.Q.T) < 1e-13


# -- pin 4: full-rank closed form ---------------------------------------------

@pytest.mark.parametrize("m,n", [(12, 20), (20, 12), (16, 16)])
def test_full_rank_closed_form(m, n):
    rng = np.random.default_rng(4)
    r = min(m, n)
    X, M, G, Q = draw(rng, m, n, r)
    res = orc.step(X, M, G, Q, MU, ETA, EPS)
    # r = min(m,n): U W^T = U U^T B = B (m <= n: U is square) or B V_basis... so M_new = mu B
    assert rel(res.M, MU * (M + G)) < 1e-12


# -- pin 5: Frobenius norm of the weight update (fixes sqrt(m/n), not n/m) ------

@pytest.mark.parametrize("m,n,r", [(24, 40, 6), (40, 24, 6)])
def test_update_norm(m, n, r):
    rng = np.random.default_rng(5)
    X, M, G, Q = draw(rng, m, n, r)
    res = orc.step(X, M, G, Q, MU, ETA, EPS)
    expect = ETA * np.sqrt(m / n) * np.sqrt(((res.d / (res.d + EPS)) ** 2).sum())
    assert abs(np.linalg.norm(res.X - X) - expect) < 1e-10 * expect
    assert abs(expect - ETA * np.sqrt(m / n) * np.sqrt(r)) < 1e-6 * expect


# -- transposed form (Section 4.3, "other variants"): invariants written out on the stored arrays --

@pytest.mark.parametrize("m,n,r", [(40, 24, 6), (24, 40, 6), (20, 20, 20), (48, 16, 16)])
def test_transposed_form_invariants(m, n, r):
    rng = np.random.default_rng(300 + m + n + r)
    X = 0.02 * rng.standard_normal((m, n)); M = rng.standard_normal((m, n)); G = rng.standard_normal((m, n))
    Q = rng.standard_normal((m, r)); Q /= np.linalg.norm(Q, axis=0)        # the warm start lives on the m side
    res = orc.step_transposed(X, M, G, Q, MU, ETA, EPS)
    B = M + G
    # the panel is B^T Q (n x r); its orthonormal factor from the library QR, sign-fixed
    q, rr = np.linalg.qr(B.T @ Q)
    U = q * np.sign(np.diag(rr))
    assert res.U.shape == (n, r) and rel(res.U, U) < 1e-10
    R = B @ U                                                              # m x r
    assert rel(res.R, R) < 1e-10
    assert rel(res.M, B - (1 - MU) * R @ U.T) < 1e-10                      # error feedback, transposed product
    d = np.linalg.norm(R, axis=0)
    assert np.allclose(res.d, d, rtol=1e-10)
    assert res.Q.shape == (m, r) and rel(res.Q, R / (d + EPS)) < 1e-10
    # the update keeps sqrt(m/n) of the stored parameter and has the transposed outer product
    assert rel(X - res.X, ETA * np.sqrt(m / n) * res.Q @ U.T) < 1e-10
    # rows of the update lie in span(U): (X - X') (I - U U^T) = 0
    D = X - res.X
    assert np.linalg.norm(D - (D @ U) @ U.T) < 1e-12 * np.linalg.norm(D)
    if r == min(m, n):
        assert rel(res.M, MU * B) < 1e-10                                  # full rank: R U^T = B


def test_transposed_form_differs_from_standard_form():
    # the two forms orthonormalize different panels: same subspace iteration target, different update
    rng = np.random.default_rng(31)
    m = n = 12; r = 3
    X, M, G, Q = draw(rng, m, n, r)
    a = orc.step(X, M, G, Q, MU, ETA, EPS)
    b = orc.step_transposed(X, M, G, Q, MU, ETA, EPS)
    assert rel(a.X, b.X) > 1e-3
    assert abs(np.linalg.norm(a.X - X) - np.linalg.norm(b.X - X)) < 1e-6 * np.linalg.norm(a.X - X)   # same scale


# -- randomized Cholesky QR (Algorithm 4) as Orthonormalize -------------------------

@pytest.mark.parametrize("m,r,decades", [(120, 24, 0), (200, 40, 6), (64, 64, 3)])
def test_rcqr_returns_the_qr_factor_whatever_the_sketch(m, r, decades):
    rng = np.random.default_rng(40 + m + r)
    P = rng.standard_normal((m, r)) @ np.diag(10.0 ** -np.linspace(0, decades, r)) @ rng.standard_normal((r, r))
    q, rr = np.linalg.qr(P)
    q = q * np.sign(np.diag(rr))                                   # library QR, positive diagonal
    k = int(np.ceil(1.25 * r))
    U1 = orc.rcqr_orthonormalize(P, rng.standard_normal((k, m)) / np.sqrt(k))
    U2 = orc.rcqr_orthonormalize(P, 7.0 * rng.standard_normal((2 * r, m)))   # other rows, other scale
    cond = np.linalg.cond(P)
    assert np.abs(U1.T @ U1 - np.eye(r)).max() < 1e-12
    assert rel(U1, q) < 1e-13 * cond and rel(U2, q) < 1e-13 * cond
    assert rel(U1 @ (U1.T @ P), P) < 1e-12                         # range(U) = range(P)
    Rq = U1.T @ P                                                  # triangular with positive diagonal
    assert np.abs(np.tril(Rq, -1)).max() < 1e-9 * np.abs(Rq).max() * max(1.0, cond * 1e-6)
    assert np.all(np.diag(Rq) > 0)


def test_step_rcqr_equals_the_plain_step():
    rng = np.random.default_rng(41)
    m, n, r = 48, 36, 9
    X, M, G, Q = draw(rng, m, n, r)
    S = rng.standard_normal((12, m)) / np.sqrt(12)
    a = orc.step(X, M, G, Q, MU, ETA, EPS)
    b = orc.step_rcqr(X, M, G, Q, S, MU, ETA, EPS)
    for name in ("X", "M", "Q", "d", "U", "R"):
        assert rel(getattr(b, name), getattr(a, name)) < 1e-11, name


# -- compressed data-parallel sync (Section 3.3): same weight update as the synchronized step ------

@pytest.mark.parametrize("ranks", [1, 2, 3])
def test_dp_sync_gives_the_update_of_the_averaged_step(ranks):
    rng = np.random.default_rng(50 + ranks)
    m, n, r = 40, 28, 7
    X, _, _, Q = draw(rng, m, n, r)
    Ms = [rng.standard_normal((m, n)) for _ in range(ranks)]
    Gs = [rng.standard_normal((m, n)) for _ in range(ranks)]
    Xn, Mn, Qn, d = orc.dp_step(X, Ms, Gs, Q, MU, ETA, EPS)
    ref = orc.step(X, sum(Ms) / ranks, sum(Gs) / ranks, Q, MU, ETA, EPS)
    assert rel(Xn, ref.X) < 1e-12 and rel(Qn, ref.Q) < 1e-12 and rel(d, ref.d) < 1e-12
    assert rel(sum(Mn) / ranks, ref.M) < 1e-12              # the mean momentum is the synchronized one
    if ranks > 1:                                           # the local momenta stay decoupled
        assert rel(Mn[0] - Mn[1], (Ms[0] + Gs[0]) - (Ms[1] + Gs[1])) < 1e-12


# -- pin 6: two-sided orthogonal equivariance (catches layout / transposition) --

def test_orthogonal_equivariance():
    rng = np.random.default_rng(6)
    m, n, r = 24, 40, 6
    X, M, G, Q = draw(rng, m, n, r)
    A, C = orth(rng, m, m), orth(rng, n, n)
    a = orc.step(X, M, G, Q, MU, ETA, EPS)
    b = orc.step(A @ X @ C.T, A @ M @ C.T, A @ G @ C.T, C @ Q, MU, ETA, EPS)
    assert rel(b.X, A @ a.X @ C.T) < 1e-12
    assert rel(b.M, A @ a.M @ C.T) < 1e-12
    assert rel(b.Q, C @ a.Q) < 1e-12


# -- pin 7: positive scale invariance -----------------------------------------

def test_scale_invariance():
    rng = np.random.default_rng(7)
    X, M, G, Q = draw(rng, 24, 40, 6)
    a = orc.step(X, M, G, Q, MU, ETA, EPS)
    b = orc.step(X, 7 * M, 7 * G, Q, MU, ETA, EPS)
    assert rel(b.X, a.X) < 1e-8 and rel(b.Q, a.Q) < 1e-8 and rel(b.M, 7 * a.M) < 1e-12


# -- pin 8: rank-1 hand case incl. the sign convention ------------------------

@pytest.mark.parametrize("flip", [1.0, -1.0])
def test_rank_one_hand_case(flip):
    rng = np.random.default_rng(8)
    m, n = 9, 14
    u = rng.standard_normal(m); u /= np.linalg.norm(u)
    v = rng.standard_normal(n); v /= np.linalg.norm(v)
    sigma = 3.5
    B = sigma * np.outer(u, v)
    q = (flip * v + 0.3 * rng.standard_normal(n))[:, None]
    sgn = np.sign(v @ q[:, 0])
    X = rng.standard_normal((m, n))
    res = orc.step(X, 0.25 * B, 0.75 * B, q, MU, ETA, 0.0)
    assert rel(res.U[:, 0], sgn * u) < 1e-13
    assert rel(res.R[:, 0], sigma * sgn * v) < 1e-13
    assert rel(res.Q[:, 0], sgn * v) < 1e-13
    assert rel(res.X, X - ETA * np.sqrt(m / n) * np.outer(u, v)) < 1e-13
    assert rel(res.M, MU * B) < 1e-13
    assert abs(res.d[0] - sigma) < 1e-13


# -- pin 9: warm-started power iteration converges to the truncated SVD --------

def test_static_buffer_converges_to_truncated_svd():
    rng = np.random.default_rng(9)
    m, n, r, k = 24, 40, 6, 8
    sig = 2.0 ** -np.arange(k)
    B0 = orth(rng, m, k) @ np.diag(sig) @ orth(rng, n, k).T
    Ub, sb, Vbt = np.linalg.svd(B0)
    polar_r = Ub[:, :r] @ Vbt[:r]
    B_r = (Ub[:, :r] * sb[:r]) @ Vbt[:r]
    Q = rng.standard_normal((n, r)); Q /= np.linalg.norm(Q, axis=0)
    errs = []
    for t in range(60):
        res = orc.step(np.zeros((m, n)), np.zeros((m, n)), B0, Q, MU, ETA, EPS)
        Q = res.Q
        O = -res.X / (ETA * np.sqrt(m / n))
        errs.append(np.linalg.norm(O - polar_r))
    floor = 10 * EPS / sig[r - 1]
    assert errs[0] > 0.1                     # not converged after one iteration from a random start
    assert errs[-1] < floor                  # converged to U_r V_r^T
    assert np.abs(res.d - sb[:r]).max() < 1e-10    # column norms -> singular values
    assert rel(res.M, B0 - (1 - MU) * B_r) < 1e-9  # error feedback keeps the residual


# -- pin 11: sign / basis facts ------------------------------------------------

def test_update_independent_of_column_signs():
    rng = np.random.default_rng(11)
    m, n, r = 24, 40, 6
    X, M, G, Q = draw(rng, m, n, r)
    res = orc.step(X, M, G, Q, MU, ETA, EPS)
    B = M + G
    sg = np.array([1, -1, 1, -1, -1, 1.0])
    U2 = res.U * sg
    R2 = B.T @ U2
    Q2 = R2 / (np.linalg.norm(R2, axis=0) + EPS)
    assert rel(B - (1 - MU) * U2 @ R2.T, res.M) < 1e-13
    assert rel(X - ETA * np.sqrt(m / n) * U2 @ Q2.T, res.X) < 1e-13
    assert rel(Q2 * sg, res.Q) < 1e-13


# -- Lazy-Dion / SymPowerIter1 (Algorithm 6) ------------------------------------

def test_sym_power_iter_and_lazy_step():
    rng = np.random.default_rng(12)
    m, n, r = 30, 20, 5
    X, M, G, Q = draw(rng, m, n, r)
    V = orc.sym_power_iter(M, Q)
    q, rr = np.linalg.qr(M.T @ (M @ Q))
    assert rel(V, q * np.sign(np.diag(rr))) < 1e-11
    for refresh in (False, True):
        Xn, Mn, Qn, d = orc.lazy_step(X, M, G, Q, MU, ETA, EPS, refresh=refresh)
        B = M + G
        Vr = orc.sym_power_iter(B, Q) if refresh else Q
        W = B @ Vr
        assert rel(Qn, Vr) < 1e-13
        assert rel(Mn, B - (1 - MU) * W @ Vr.T) < 1e-13
        assert np.allclose(d, np.linalg.norm(W, axis=0), rtol=1e-13)
        assert rel(Xn, X - ETA * np.sqrt(m / n) * (W / (d + EPS)) @ Vr.T) < 1e-13
    # with an orthonormal V the lazy error feedback is a projector: M_new V = mu B V
    Xn, Mn, Qn, d = orc.lazy_step(X, M, G, Q, MU, ETA, EPS, refresh=True)
    assert rel(Mn @ Qn, MU * (M + G) @ Qn) < 1e-12


def test_lazy_step_update_norm_with_orthonormal_right_factor():
    # after a refresh V is orthonormal, so ||ColNorm(W) V^T||_F = ||ColNorm(W)||_F: the update has
    # norm eta sqrt(m/n) sqrt(sum_j (d_j / (d_j + eps))^2), whatever W is (fixes the scale factor,
    # the use of the normalised W and of V in the update of Algorithm 6)
    rng = np.random.default_rng(21)
    for m, n, r in ((30, 20, 5), (18, 44, 7)):
        X, M, G, Q = draw(rng, m, n, r)
        Xn, Mn, Qn, d = orc.lazy_step(X, M, G, Q, MU, ETA, EPS, refresh=True)
        assert rel(Qn.T @ Qn, np.eye(r)) < 1e-12
        want = ETA * np.sqrt(m / n) * np.sqrt(np.sum((d / (d + EPS)) ** 2))
        assert abs(np.linalg.norm(Xn - X) - want) < 1e-9 * want
        assert abs(want - ETA * np.sqrt(m / n) * np.sqrt(r)) < 1e-6 * want
        # the update lies in span(V) on the right: (X - X_new) (I - V V^T) = 0
        D = X - Xn
        assert np.linalg.norm(D - D @ Qn @ Qn.T) < 1e-12 * np.linalg.norm(D)


def test_lazy_dion_with_refresh_every_step_converges_to_truncated_svd():
    # Lazy-Dion_k with k = 1 on a static buffer: V <- Orthonormalize(B^T B V) is orthogonal iteration,
    # so V -> V_r column by column, W = B V -> U_r Sigma_r, ColNorm(W) V^T -> U_r V_r^T, d -> sigma and
    # M_new -> B - beta B_r, against a brute-force SVD
    rng = np.random.default_rng(22)
    m, n, r, k = 24, 40, 6, 8
    sig = 2.0 ** -np.arange(k)
    B0 = orth(rng, m, k) @ np.diag(sig) @ orth(rng, n, k).T
    Ub, sb, Vbt = np.linalg.svd(B0)
    polar_r = Ub[:, :r] @ Vbt[:r]
    B_r = (Ub[:, :r] * sb[:r]) @ Vbt[:r]
    Q = rng.standard_normal((n, r)); Q /= np.linalg.norm(Q, axis=0)
    errs = []
    for t in range(40):
        Xn, Mn, Q, d = orc.lazy_step(np.zeros((m, n)), np.zeros((m, n)), B0, Q, MU, ETA, EPS, refresh=True)
        O = -Xn / (ETA * np.sqrt(m / n))
        errs.append(np.linalg.norm(O - polar_r))
    assert errs[0] > 0.1
    assert errs[-1] < 10 * EPS / sig[r - 1]
    assert np.abs(d - sb[:r]).max() < 1e-10
    assert rel(Mn, B0 - (1 - MU) * B_r) < 1e-9


def test_row_sampled_step_equals_the_full_step_on_those_rows():
    rng = np.random.default_rng(23)
    m, n, r = 37, 29, 9
    X, M, G, Q = draw(rng, m, n, r)
    res = orc.step(X, M, G, Q, MU, ETA, EPS)
    rows = np.array([0, 5, 36, 17, 5])
    Xr, Mr, Qn, d = orc.step_rows(X, M, G, Q, rows, MU, ETA, EPS)
    assert rel(Xr, res.X[rows]) < 1e-13 and rel(Mr, res.M[rows]) < 1e-13
    assert rel(Qn, res.Q) < 1e-13 and rel(d, res.d) < 1e-13


def test_step_given_panel_is_the_step_when_the_panel_is_exact():
    rng = np.random.default_rng(24)
    m, n, r = 33, 21, 8
    X, M, G, Q = draw(rng, m, n, r)
    res = orc.step(X, M, G, Q, MU, ETA, EPS)
    alt = orc.step_given_panel(X, M, G, Q, (M + G) @ Q, MU, ETA, EPS)
    for a, b in ((alt.X, res.X), (alt.M, res.M), (alt.Q, res.Q), (alt.d, res.d), (alt.U, res.U)):
        assert rel(a, b) < 1e-12
    # a scaled panel has the same thin-QR factor: the outputs do not move
    alt2 = orc.step_given_panel(X, M, G, Q, 3.0 * ((M + G) @ Q), MU, ETA, EPS)
    assert rel(alt2.X, res.X) < 1e-12 and rel(alt2.Q, res.Q) < 1e-12


@pytest.mark.parametrize("ranks,m,n,r", [(2, 20, 30, 6), (3, 17, 31, 5), (4, 12, 16, 8), (1, 9, 7, 3)])
def test_sharded_step_equals_the_centralised_step_layer_by_layer(ranks, m, n, r):
    # Algorithm 3 is built to preserve the mathematics of Algorithm 2: whatever the number of column shards
    # (ragged ones and shards narrower than r included), every layer must come out as the unsharded step
    rng = np.random.default_rng(30 + ranks)
    layers = [draw(rng, m, n, r) for _ in range(ranks)]
    Xs, Ms, Gs, Qs = (list(t) for t in zip(*layers))
    Xn, Mn, Vn, d = orc.sharded_step(Xs, Ms, Gs, Qs, MU, ETA, EPS)
    for l in range(ranks):
        res = orc.step(Xs[l], Ms[l], Gs[l], Qs[l], MU, ETA, EPS)
        assert rel(Xn[l], res.X) < 1e-12 and rel(Mn[l], res.M) < 1e-12
        assert rel(Vn[l], res.Q) < 1e-12 and rel(d[l], res.d) < 1e-12
    bounds = orc.shard_bounds(n, ranks)
    assert bounds[0][0] == 0 and bounds[-1][1] == n and all(a[1] == b[0] for a, b in zip(bounds, bounds[1:]))


# -- generated benchmark inputs are in contract ---------------------------------

def test_config1_ten_steps_stay_in_contract():
    import torch
    from paper_2504_05295_b200 import inputs
    m, n, r, ks = inputs.config1()
    pb = inputs.make_problem(m, n, r, seed=0, ks=ks)
    X, M, Q = pb.X.double().numpy(), pb.M.double().numpy(), pb.Q.double().numpy()
    assert np.allclose(np.linalg.norm(Q, axis=0), 1.0, atol=1e-6)
    assert rel(pb.Us.double().numpy().T @ pb.Us.double().numpy(), np.eye(ks)) < 1e-5
    for t in range(10):
        G = pb.grad(t).double().numpy()
        res = orc.step(X, M, G, Q, MU, ETA, EPS)
        assert res.degenerate == 0
        assert np.linalg.cond(res.P) < 50          # CholeskyQR-safe at rank fraction 1/4
        X, M, Q = res.X, res.M, res.Q
    assert np.all(np.isfinite(X)) and res.d.min() > 1.0

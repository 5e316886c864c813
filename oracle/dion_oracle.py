"""ctypes front end of the float64 CPU oracle (``dion_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports or links this.

Every function takes and returns C-contiguous float64 numpy arrays.  State
arrays are copied, so callers keep their inputs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import NamedTuple, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dion_oracle.c")


def _cpu_tag() -> str:
    """Short hash of this host's CPU feature flags: the library is compiled with
    -march=native, so a copy built on another machine must not be reused."""
    import hashlib
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.sha1(flags.encode()).hexdigest()[:10]


_LIB = os.path.join(_HERE, f"libdion_oracle_{_cpu_tag()}.so")

_i64 = ctypes.c_int64
_dbl = ctypes.c_double
_ptr = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O3 -fopenmp).  Returns the library path."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11",
           "-fno-fast-math", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True, capture_output=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.dion_oracle_num_threads.restype = ctypes.c_int
        lib.dion_oracle_householder_qr.restype = ctypes.c_int
        lib.dion_oracle_householder_qr.argtypes = [_i64, _i64, _ptr, _ptr, _ptr]
        lib.dion_oracle_colnorm.restype = None
        lib.dion_oracle_colnorm.argtypes = [_i64, _i64, _ptr, _dbl, _ptr]
        lib.dion_oracle_step.restype = ctypes.c_int
        lib.dion_oracle_step.argtypes = [_i64, _i64, _i64, _ptr, _ptr, _ptr, _ptr,
                                         _dbl, _dbl, _dbl, _ptr, _ptr, _ptr, _ptr]
        lib.dion_oracle_sym_power_iter.restype = ctypes.c_int
        lib.dion_oracle_sym_power_iter.argtypes = [_i64, _i64, _i64, _ptr, _ptr]
        lib.dion_oracle_lazy_step.restype = ctypes.c_int
        lib.dion_oracle_lazy_step.argtypes = [_i64, _i64, _i64, _ptr, _ptr, _ptr, _ptr,
                                              _dbl, _dbl, _dbl, ctypes.c_int, _ptr]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().dion_oracle_num_threads())


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_ptr)


class StepResult(NamedTuple):
    X: np.ndarray      # m x n, updated parameter
    M: np.ndarray      # m x n, updated momentum
    Q: np.ndarray      # n x r, updated right factor (the paper's V_new)
    d: np.ndarray      # r, column norms of W (singular value estimates)
    P: np.ndarray      # m x r, B V before orthonormalization
    U: np.ndarray      # m x r, orthonormal left factor
    R: np.ndarray      # n x r, the paper's W = B^T U
    degenerate: int    # number of degenerate Householder columns


def householder_qr(P):
    """Thin QR with diag(R) >= 0.  Returns (U, R_qr)."""
    P = _f64(P)
    m, r = P.shape
    U = np.empty((m, r))
    Rqr = np.empty((r, r))
    rc = _load().dion_oracle_householder_qr(m, r, _p(P), _p(U), _p(Rqr))
    if rc < 0:
        raise MemoryError("oracle: out of host memory")
    return U, Rqr


def colnorm(W, eps: float):
    W = _f64(W).copy()
    n, r = W.shape
    d = np.empty(r)
    _load().dion_oracle_colnorm(n, r, _p(W), float(eps), _p(d))
    return W, d


def step(X, M, G, Q, mu: float, eta: float, eps: float = 1e-8) -> StepResult:
    """One Dion step (Algorithm 1 + 2).  Inputs are not modified."""
    X = _f64(X).copy(); M = _f64(M).copy(); G = _f64(G); Q = _f64(Q).copy()
    m, n = X.shape
    r = Q.shape[1]
    assert M.shape == (m, n) and G.shape == (m, n) and Q.shape == (n, r)
    assert 1 <= r <= min(m, n)
    d = np.empty(r); P = np.empty((m, r)); U = np.empty((m, r)); R = np.empty((n, r))
    rc = _load().dion_oracle_step(m, n, r, _p(X), _p(M), _p(G), _p(Q), float(mu), float(eta),
                                  float(eps), _p(d), _p(P), _p(U), _p(R))
    if rc < 0:
        raise MemoryError("oracle: out of host memory")
    return StepResult(X, M, Q, d, P, U, R, rc)


def step_rows(X, M, G, Q, rows, mu: float, eta: float, eps: float = 1e-8):
    """The Dion step (Algorithm 1 + 2) with its two m x n outputs formed for the given
    rows only, for matrices too large to run ``step`` on: B = M + G; P = B V; U = Householder
    thin-QR factor of P (positive diagonal); W = B^T U; V_new = ColNorm(W); then, for each
    requested row i, M_new[i] = B[i] - (1 - mu) U[i] W^T and X_new[i] = X[i] - eta sqrt(m/n)
    U[i] V_new^T.  The factors are those of the whole matrix; only the rank-r outer products
    are restricted to the rows.  The two large contractions are library matrix products in
    float64.  Returns (X_rows, M_rows, V_new, d)."""
    X = _f64(X); M = _f64(M); G = _f64(G); Q = _f64(Q)
    m, n = X.shape
    rows = np.asarray(rows, dtype=np.int64)
    B = M + G
    P = B @ Q
    U, _ = householder_qr(P)
    W = B.T @ U
    Qn, d = colnorm(W, eps)
    Ur = U[rows]
    Mr = B[rows] - (1.0 - mu) * (Ur @ W.T)
    Xr = X[rows] - eta * np.sqrt(m / n) * (Ur @ Qn.T)
    return Xr, Mr, Qn, d


def step_given_panel(X, M, G, Q, P, mu: float, eta: float, eps: float = 1e-8) -> StepResult:
    """The Dion step (Algorithm 1 + 2) from PowerIter1's second line on, with the panel P handed in
    by the caller instead of being formed as B V: U = Householder thin-QR factor of P, W = B^T U,
    M_new = B - (1 - mu) U W^T, V_new = ColNorm(W), X_new = X - eta sqrt(m/n) U V_new^T.
    With P = (M + G) Q it is ``step``.  Tests use it to measure how far the float64 rule itself moves
    when P carries the rounding error of a float32 product (the rule's own conditioning)."""
    X = _f64(X); M = _f64(M); G = _f64(G); Q = _f64(Q); P = _f64(P)
    m, n = X.shape
    B = M + G
    U, _ = householder_qr(P)
    W = B.T @ U
    Qn, d = colnorm(W, eps)
    Mn = B - (1.0 - mu) * (U @ W.T)
    Xn = X - eta * np.sqrt(m / n) * (U @ Qn.T)
    return StepResult(Xn, Mn, Qn, d, P, U, W, 0)


def step_transposed(X, M, G, Q, mu: float, eta: float, eps: float = 1e-8) -> StepResult:
    """One Dion step in the transposed form (Section 4.3, "other variants": the power
    iteration runs on M^T).  By definition this is the standard step on the transposed
    arrays, X^T, M^T, G^T (n x m) with Q of shape m x r.  The update keeps the factor
    sqrt(m/n) of the stored m x n parameter (rows = "out"): the standard step on the
    n x m arrays applies sqrt(n/m), so it is given eta * m / n.
    Returns X, M (m x n again), Q (m x r), d, and P, U (n x r), R (m x r)."""
    X = _f64(X); M = _f64(M); G = _f64(G)
    m, n = X.shape
    res = step(np.ascontiguousarray(X.T), np.ascontiguousarray(M.T), np.ascontiguousarray(G.T), Q,
               mu, float(eta) * m / n, eps)
    return StepResult(np.ascontiguousarray(res.X.T), np.ascontiguousarray(res.M.T), res.Q, res.d,
                      res.P, res.U, res.R, res.degenerate)


def rcqr_orthonormalize(P, S):
    """Distributed-Orthonormalize (Algorithm 4) on one device, step by step in float64:
    sketch Pt = S P; R1 = triangular factor of QR(Pt); B = P R1^-1; R2 = Cholesky(B^T B)
    (upper factor); U = B R2^-1.  S is the caller's sketching matrix (k x m, k >= r).
    The signs of R1 are normalised to a positive diagonal, so U is the thin-QR factor of P
    with positive diagonal whatever S is."""
    P = _f64(P); S = _f64(S)
    m, r = P.shape
    assert S.shape[1] == m and S.shape[0] >= r
    Pt = S @ P
    R1 = np.linalg.qr(Pt, mode="r")
    R1 = R1 * np.sign(np.diag(R1))[:, None]
    B = np.linalg.solve(R1.T, P.T).T            # B R1 = P
    G = B.T @ B
    R2 = np.linalg.cholesky(G).T                # G = R2^T R2
    U = np.linalg.solve(R2.T, B.T).T            # U R2 = B
    return U


def step_rcqr(X, M, G, Q, S, mu: float, eta: float, eps: float = 1e-8) -> StepResult:
    """One Dion step (Algorithm 1 + 2) whose Orthonormalize is Algorithm 4 with sketch S."""
    X = _f64(X); M = _f64(M); G = _f64(G); Q = _f64(Q)
    m, n = X.shape
    B = M + G
    P = B @ Q
    U = rcqr_orthonormalize(P, S)
    R = B.T @ U
    Mn = B - (1.0 - mu) * (U @ R.T)
    d = np.sqrt((R * R).sum(axis=0))
    Qn = R / (d + eps)
    Xn = X - eta * np.sqrt(m / n) * (U @ Qn.T)
    return StepResult(Xn, Mn, Qn, d, P, U, R, 0)


def dp_step(X, Ms, Gs, Q, mu: float, eta: float, eps: float = 1e-8):
    """One Dion step with compressed data-parallel sync (Section 3.3; the AllReduce lines of
    PowerIter1): rank i holds its own momentum Ms[i] and gradient Gs[i], all ranks hold X and Q.
    P and W are averaged over the ranks; each momentum takes the same low-rank correction.
    Returns (X, [M_i], Q, d)."""
    X = _f64(X); Q = _f64(Q)
    Bs = [_f64(M) + _f64(G) for M, G in zip(Ms, Gs)]
    m, n = X.shape
    P = sum(B @ Q for B in Bs) / len(Bs)                     # AllReduce (mean) of the local B_i V
    U, _ = householder_qr(P)                                 # Orthonormalize: thin QR, positive diagonal
    W = sum(B.T @ U for B in Bs) / len(Bs)                   # AllReduce (mean) of the local B_i^T U
    d = np.sqrt((W * W).sum(axis=0))
    Qn = W / (d + eps)
    Mn = [B - (1.0 - mu) * (U @ W.T) for B in Bs]
    Xn = X - eta * np.sqrt(m / n) * (U @ Qn.T)
    return Xn, Mn, Qn, d


def shard_bounds(n: int, ranks: int):
    """Contiguous column blocks J_0, ..., J_{ranks-1} of 0..n-1 (the first n % ranks blocks one longer)."""
    base, extra = divmod(n, ranks)
    out, lo = [], 0
    for x in range(ranks):
        hi = lo + base + (1 if x < extra else 0)
        out.append((lo, hi))
        lo = hi
    return out


def sharded_step(X, M, G, Q, mu: float, eta: float, eps: float = 1e-8):
    """1D-sharded Dion (Algorithm 3) on L layers of identical shape over |X| = L ranks, emulated rank by rank.
    X, M, G: lists of L arrays (m x n); Q: list of L arrays (n x r).  Rank x holds the columns J_x of every layer's
    X, M, G and the rows J_x of every layer's V; what it computes below uses only those (and what the
    collectives hand it).  The lines follow the algorithm:
      1  B = M + G on the local shards
      2  partial P_x[l] = B[l][:, J_x] V[l][J_x, :]                        (unreduced over the ranks)
      3  ReduceScatter along L: rank l receives P[l] = sum_x P_x[l]
      4  rank l: U[l] = Orthonormalize(P[l])  (Householder thin QR, positive diagonal)
      5  AllGather: every rank holds U[l] for all l
      6  W_x[l] = B[l][:, J_x]^T U[l]                                      (rows J_x of W[l])
      7  M_new[l][:, J_x] = B[l][:, J_x] - (1 - mu) U[l] W_x[l]^T
      8  ColNorm with an AllReduce(sum) of the squared column norms over the ranks
      9  O = U V_new^T on the shard; X_new = X - eta sqrt(m/n) O with n the full number of columns.
    Returns (X_new, M_new, V_new, d): lists of L full arrays reassembled from the shards."""
    L = len(X)
    X = [_f64(a) for a in X]; M = [_f64(a) for a in M]; G = [_f64(a) for a in G]; Q = [_f64(a) for a in Q]
    m, n = X[0].shape
    r = Q[0].shape[1]
    J = shard_bounds(n, L)
    B = [[M[l][:, lo:hi] + G[l][:, lo:hi] for l in range(L)] for (lo, hi) in J]          # B[x][l]: rank x, layer l
    Ppart = [[B[x][l] @ Q[l][J[x][0]:J[x][1], :] for l in range(L)] for x in range(L)]
    P = [sum(Ppart[x][l] for x in range(L)) for l in range(L)]                           # rank l owns P[l]
    U = [householder_qr(P[l])[0] for l in range(L)]
    W = [[B[x][l].T @ U[l] for l in range(L)] for x in range(L)]
    sumsq = [sum((W[x][l] * W[x][l]).sum(axis=0) for x in range(L)) for l in range(L)]   # AllReduce of r scalars per layer
    d = [np.sqrt(sq) for sq in sumsq]
    Xn = [np.empty((m, n)) for _ in range(L)]
    Mn = [np.empty((m, n)) for _ in range(L)]
    Vn = [np.empty((n, r)) for _ in range(L)]
    for x, (lo, hi) in enumerate(J):
        for l in range(L):
            Vx = W[x][l] / (d[l] + eps)
            Mn[l][:, lo:hi] = B[x][l] - (1.0 - mu) * (U[l] @ W[x][l].T)
            Xn[l][:, lo:hi] = X[l][:, lo:hi] - eta * np.sqrt(m / n) * (U[l] @ Vx.T)
            Vn[l][lo:hi, :] = Vx
    return Xn, Mn, Vn, d


def sym_power_iter(M, Q):
    """SymPowerIter1 (Algorithm 6): Orthonormalize(M^T M V)."""
    M = _f64(M); Q = _f64(Q).copy()
    m, n = M.shape
    r = Q.shape[1]
    rc = _load().dion_oracle_sym_power_iter(m, n, r, _p(M), _p(Q))
    if rc < 0:
        raise MemoryError("oracle: out of host memory")
    return Q


def lazy_step(X, M, G, Q, mu: float, eta: float, eps: float = 1e-8, refresh: bool = False):
    """One Lazy-Dion step (Algorithm 6).  Returns (X, M, Q, d)."""
    X = _f64(X).copy(); M = _f64(M).copy(); G = _f64(G); Q = _f64(Q).copy()
    m, n = X.shape
    r = Q.shape[1]
    d = np.empty(r)
    rc = _load().dion_oracle_lazy_step(m, n, r, _p(X), _p(M), _p(G), _p(Q), float(mu), float(eta),
                                       float(eps), int(bool(refresh)), _p(d))
    if rc < 0:
        raise MemoryError("oracle: out of host memory")
    return X, M, Q, d


if __name__ == "__main__":
    print(build(force=True))

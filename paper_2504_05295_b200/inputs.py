"""Seeded synthetic inputs for the Dion step.

This module is the only code shared by the CPU oracle's tests and the CUDA
path's tests and benchmark.  It holds none of the method's arithmetic: it
draws parameters, optimizer state and gradients with the statistics of the
benchmark configurations and returns plain ``torch`` tensors.  The same bytes
are handed to both sides; nothing depends on matching random streams between
host and device.

Recipe (per matrix ``k`` of a workload, ``seed_k = 1000003 * seed + k``):

* ``X ~ N(0, 0.02^2)``, ``M = 0``, ``Q0 ~ N(0, 1)`` with every column scaled to
  unit 2-norm, all fp32;
* a fixed low-rank signal ``S = Us diag(s) Vs^T`` with ``Us`` (m x ks) and ``Vs``
  (n x ks) the orthonormal factors of Gaussian matrices, ``s_i = 2^(-i/2)``,
  ``i = 0 .. ks-1``; drawn once per matrix;
* per step ``t``: ``G_t = S + 0.1 * Z_t`` with ``Z_t ~ N(0, 1)`` fresh, rounded once
  to the gradient's storage type (fp32, or bf16 round-to-nearest-even).

The signal stands in for the slowly drifting dominant subspace of a real
momentum buffer; the noise keeps the projected panel ``P`` well conditioned at
rank fractions <= 1/4 and ill conditioned (1e4 .. 1e6) at full rank.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional, Tuple

import torch

SEED_STRIDE = 1000003


def matrix_seed(seed: int, k: int) -> int:
    return SEED_STRIDE * int(seed) + int(k)


def rank_from_fraction(m: int, n: int, fraction: float) -> int:
    """r = max(1, floor(fraction * min(m, n)))."""
    return max(1, int(fraction * min(m, n)))


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn(shape, gen: torch.Generator, device) -> torch.Tensor:
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)


def _orthonormal_columns(rows: int, cols: int, gen: torch.Generator, device) -> torch.Tensor:
    """Orthonormal basis of a Gaussian (rows x cols) matrix, signs fixed so the
    triangular factor has a positive diagonal (input generation only)."""
    a = _randn((rows, cols), gen, device).double()
    q, rr = torch.linalg.qr(a, mode="reduced")
    sgn = torch.sign(torch.diagonal(rr))
    sgn[sgn == 0] = 1.0
    return (q * sgn).float()


@dataclass
class DionProblem:
    """State and gradient source of one matrix parameter."""
    m: int
    n: int
    r: int
    X: torch.Tensor          # m x n fp32
    M: torch.Tensor          # m x n fp32 (zeros)
    Q: torch.Tensor          # n x r fp32, unit-norm columns
    S: Optional[torch.Tensor]  # m x n fp32 low-rank signal (None when only factors are kept)
    Us: torch.Tensor         # m x ks
    Vs: torch.Tensor         # n x ks
    s: torch.Tensor          # ks
    seed: int
    g_dtype: torch.dtype
    noise: float = 0.1

    def grad(self, step: int, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Gradient of step ``step`` (0-based): signal + fresh Gaussian noise,
        rounded once to ``g_dtype``."""
        dev = self.X.device
        gen = _gen(matrix_seed(self.seed, 7919 * (step + 1)), dev)
        z = _randn((self.m, self.n), gen, dev)
        z.mul_(self.noise)
        if self.S is not None:
            z.add_(self.S)
        else:
            z.addmm_(self.Us * self.s, self.Vs.t())
        g = z.to(self.g_dtype)
        if out is not None:
            out.copy_(g)
            return out
        return g


def make_problem(m: int, n: int, r: int, seed: int = 0, k: int = 0, ks: int = 64,
                 g_dtype: torch.dtype = torch.float32, device="cpu",
                 keep_signal: bool = True) -> DionProblem:
    """Draw X, M = 0, Q0 and the fixed signal of matrix ``k`` of a workload."""
    assert 1 <= r <= min(m, n)
    ks = min(ks, m, n)
    sk = matrix_seed(seed, k)
    gen = _gen(sk, device)
    X = _randn((m, n), gen, device).mul_(0.02)
    M = torch.zeros((m, n), dtype=torch.float32, device=device)
    Q = _randn((n, r), gen, device)
    Q = (Q / torch.linalg.vector_norm(Q.double(), dim=0).float()).contiguous()
    Us = _orthonormal_columns(m, ks, gen, device)
    Vs = _orthonormal_columns(n, ks, gen, device)
    s = torch.pow(2.0, -0.5 * torch.arange(ks, dtype=torch.float32, device=device))
    S = ((Us * s) @ Vs.t()).contiguous() if keep_signal else None
    return DionProblem(m, n, r, X, M, Q, S, Us, Vs, s, sk, g_dtype)


def row_side_factor(pb: DionProblem, device=None) -> torch.Tensor:
    """Warm-start factor of the transposed form: m x r, unit-norm Gaussian columns,
    drawn from the matrix's own seed (independent of its n x r factor)."""
    dev = pb.X.device if device is None else device
    gen = _gen(matrix_seed(pb.seed, 104729), dev)
    Q = _randn((pb.m, pb.r), gen, dev)
    return (Q / torch.linalg.vector_norm(Q.double(), dim=0).float()).contiguous()


def sketch_matrix(pb: DionProblem, rows: Optional[int] = None, transposed: bool = False, device=None) -> torch.Tensor:
    """Sketching matrix of the randomized Cholesky QR (Algorithm 4): `rows` x p Gaussian entries of
    standard deviation 1/sqrt(rows), p = the number of panel rows (m, or n in the transposed form);
    rows defaults to ceil(1.25 r).  Drawn from the matrix's own seed."""
    dev = pb.X.device if device is None else device
    k = int(math.ceil(1.25 * pb.r)) if rows is None else int(rows)
    p = pb.n if transposed else pb.m
    gen = _gen(matrix_seed(pb.seed, 15485863), dev)
    return (_randn((k, p), gen, dev) / math.sqrt(k)).contiguous()


# ---------------------------------------------------------------------------
# The benchmark configurations (shapes only; tensors are drawn by make_problem)
# ---------------------------------------------------------------------------

def config1() -> Tuple[int, int, int, int]:
    """Single fp32 matrix 256 x 512, r = 64, signal rank 16."""
    return 256, 512, 64, 16


def config2_cases() -> List[Tuple[int, int, int]]:
    """Square fp32 matrices 2048^2, 4096^2, 8192^2 at rank fractions 1, 1/4, 1/16."""
    out = []
    for d in (2048, 4096, 8192):
        for f in (1.0, 0.25, 0.0625):
            out.append((d, d, rank_from_fraction(d, d, f)))
    return out


def config3_cases() -> List[Tuple[int, int, int]]:
    """16384^2 and 32768^2 at rank fractions 1/4, 1/16, 1/64."""
    out = []
    for d in (16384, 32768):
        for f in (0.25, 0.0625, 0.015625):
            out.append((d, d, rank_from_fraction(d, d, f)))
    return out


def llama_block_shapes(hidden: int, kv: int, ffn: int) -> List[Tuple[str, int, int]]:
    """(name, m, n) of the seven matrices of one transformer block, rows = out."""
    return [("q", hidden, hidden), ("k", kv, hidden), ("v", kv, hidden), ("o", hidden, hidden),
            ("gate", ffn, hidden), ("up", ffn, hidden), ("down", hidden, ffn)]


def config4_shapes(layers: int = 32) -> List[Tuple[str, int, int]]:
    """Llama-3-8B-shaped list: ``layers`` blocks of seven matrices."""
    out = []
    for l in range(layers):
        out += [(f"l{l}.{nm}", m, n) for nm, m, n in llama_block_shapes(4096, 1024, 14336)]
    return out


def config5_shapes() -> List[Tuple[str, int, int]]:
    """Llama-3-405B-shaped single block."""
    return llama_block_shapes(16384, 1024, 53248)

"""Shared helpers of the parity tests: run the same seeded inputs through the
CPU oracle and through the CUDA library (C-ABI via the ctypes binding)."""
from __future__ import annotations

import numpy as np
import torch

from oracle import dion_oracle as orc
from paper_2504_05295_b200 import inputs

MU, ETA, EPS = 0.95, 0.01, 1e-8
TOL_FP32 = 1e-4   # relative Frobenius error on X, M, Q, fp32 path
TOL_BF16 = 3e-2   # bf16-operand path


def rel(a, b) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def oracle_steps(pb: inputs.DionProblem, steps: int, grads=None, mu=MU, eta=ETA, eps=EPS):
    """Float64 oracle over `steps` steps; state carried in float64.  Returns the
    list of StepResult (one per step)."""
    X, M, Q = to_np64(pb.X), to_np64(pb.M), to_np64(pb.Q)
    out = []
    for t in range(steps):
        G = to_np64(grads[t] if grads is not None else pb.grad(t))
        res = orc.step(X, M, G, Q, mu, eta, eps)
        X, M, Q = res.X, res.M, res.Q
        out.append(res)
    return out


def device_state(pb: inputs.DionProblem, dev="cuda"):
    return (pb.X.to(dev).clone(), pb.M.to(dev).clone(), pb.Q.to(dev).clone())

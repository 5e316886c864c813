"""Thin ctypes binding of ``libdion_b200.so`` (the C-ABI declared in ``include/dion.h``).

Argument marshalling only: every arithmetic step runs in the CUDA kernels.
PyTorch supplies device memory and streams.  There is no CPU or eager-PyTorch
fallback: if the shared library is missing or no sm_100 device is present the
calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Iterable, List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdion_b200.so")

DION_F32, DION_BF16 = 0, 1
PREC_FP32, PREC_BF16_OPERANDS = 0, 1
ORTH_AUTO, ORTH_CHOLQR2, ORTH_SHIFTED3, ORTH_HOUSEHOLDER, ORTH_RCQR = 0, 1, 2, 3, 4
ENGINE_AUTO, ENGINE_SIMT, ENGINE_TENSOR = 0, 1, 2
STATUS_BREAKDOWN, STATUS_NONFINITE, STATUS_TIMEOUT, STATUS_ILLCOND = 1, 2, 4, 8

EXPORTS = ["dion_default_config", "dion_init", "dion_step", "dion_step_grouped", "dion_lazy_step",
           "dion_workspace_bytes", "dion_get_status", "dion_launch_count", "dion_destroy",
           "dion_strerror", "dion_profile_enable", "dion_profile_read", "dion_get_orth_rounds", "dion_get_fallbacks",
           "dion_step_noalloc", "dion_noalloc_scratch_limit", "dion_dp_project", "dion_dp_factor",
           "dion_dp_finish", "dion_shard_project", "dion_orthonormalize", "dion_shard_factor", "dion_shard_finish"]
PHASES = ["P", "ORTH", "R", "EF", "COLNORM", "X", "ORTH_GEMM"]


class DionConfig(ctypes.Structure):
    _fields_ = [("mu", ctypes.c_float), ("eps", ctypes.c_float), ("precision", ctypes.c_int),
                ("orth", ctypes.c_int), ("engine", ctypes.c_int), ("device", ctypes.c_int),
                ("workspace_bytes", ctypes.c_size_t)]


class DionMatrix(ctypes.Structure):
    _fields_ = [("m", ctypes.c_int64), ("n", ctypes.c_int64), ("r", ctypes.c_int64),
                ("X", ctypes.c_void_p), ("ldx", ctypes.c_int64),
                ("M", ctypes.c_void_p), ("ldm", ctypes.c_int64),
                ("G", ctypes.c_void_p), ("ldg", ctypes.c_int64), ("g_dtype", ctypes.c_int),
                ("Q", ctypes.c_void_p), ("ldq", ctypes.c_int64),
                ("colnorm_out", ctypes.c_void_p), ("transposed", ctypes.c_int),
                ("sketch", ctypes.c_void_p), ("sketch_rows", ctypes.c_int64), ("ld_sketch", ctypes.c_int64)]


class DionError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"dion error {code}: {msg}")
        self.code = code


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2504_05295_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64, f32, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_float, ctypes.c_int
    lib.dion_default_config.argtypes = [ctypes.POINTER(DionConfig)]
    lib.dion_default_config.restype = None
    lib.dion_init.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(DionConfig)]
    lib.dion_init.restype = ci
    lib.dion_step.argtypes = [vp, ctypes.POINTER(DionMatrix), f32, vp]
    lib.dion_step.restype = ci
    lib.dion_step_grouped.argtypes = [vp, ctypes.POINTER(DionMatrix), ci, f32, vp]
    lib.dion_step_grouped.restype = ci
    lib.dion_lazy_step.argtypes = [vp, ctypes.POINTER(DionMatrix), f32, ci, vp]
    lib.dion_lazy_step.restype = ci
    lib.dion_workspace_bytes.argtypes = [vp, i64, i64, i64]
    lib.dion_workspace_bytes.restype = ctypes.c_size_t
    lib.dion_get_status.argtypes = [vp, vp, ctypes.POINTER(ci), ctypes.POINTER(ci)]
    lib.dion_get_status.restype = ci
    lib.dion_launch_count.argtypes = [vp]
    lib.dion_launch_count.restype = i64
    lib.dion_profile_enable.argtypes = [vp, ci]
    lib.dion_profile_enable.restype = ci
    lib.dion_profile_read.argtypes = [vp, ctypes.POINTER(f32), ctypes.POINTER(i64)]
    lib.dion_profile_read.restype = ci
    lib.dion_get_orth_rounds.argtypes = [vp, vp, ctypes.POINTER(i64)]
    lib.dion_get_orth_rounds.restype = ci
    lib.dion_get_fallbacks.argtypes = [vp, vp, ctypes.POINTER(i64)]
    lib.dion_get_fallbacks.restype = ci
    lib.dion_step_noalloc.argtypes = [ctypes.POINTER(DionMatrix), f32, f32, f32, vp]
    lib.dion_step_noalloc.restype = ci
    lib.dion_noalloc_scratch_limit.argtypes = []
    lib.dion_noalloc_scratch_limit.restype = ctypes.c_size_t
    lib.dion_dp_project.argtypes = [vp, ctypes.POINTER(DionMatrix), vp, vp, vp]
    lib.dion_dp_project.restype = ci
    lib.dion_dp_factor.argtypes = [vp, ctypes.POINTER(DionMatrix), vp, vp, vp, vp]
    lib.dion_dp_factor.restype = ci
    lib.dion_dp_finish.argtypes = [vp, ctypes.POINTER(DionMatrix), vp, vp, vp, f32, vp]
    lib.dion_dp_finish.restype = ci
    lib.dion_shard_project.argtypes = [vp, ctypes.POINTER(DionMatrix), i64, vp, vp, vp]
    lib.dion_shard_project.restype = ci
    lib.dion_orthonormalize.argtypes = [vp, i64, i64, i64, vp, vp, vp]
    lib.dion_orthonormalize.restype = ci
    lib.dion_shard_factor.argtypes = [vp, ctypes.POINTER(DionMatrix), i64, vp, vp, vp, vp, vp]
    lib.dion_shard_factor.restype = ci
    lib.dion_shard_finish.argtypes = [vp, ctypes.POINTER(DionMatrix), i64, vp, vp, vp, vp, f32, vp]
    lib.dion_shard_finish.restype = ci
    lib.dion_destroy.argtypes = [vp]
    lib.dion_destroy.restype = None
    lib.dion_strerror.argtypes = [ci]
    lib.dion_strerror.restype = ctypes.c_char_p
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().dion_strerror(int(code)).decode()


def _check(code: int) -> None:
    if code != 0:
        raise DionError(code, strerror(code))


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def matrix_desc(X: torch.Tensor, M: torch.Tensor, G: torch.Tensor, Q: torch.Tensor,
                colnorm_out: Optional[torch.Tensor] = None, transposed: bool = False,
                sketch: Optional[torch.Tensor] = None) -> DionMatrix:
    """Describes one parameter for the C-ABI.  Tensors must be CUDA, 2-D, row-major
    (unit stride along the last dimension); a row stride larger than the width is
    passed on as the leading dimension.  Q is n x r, or m x r in the transposed form."""
    for name, t in (("X", X), ("M", M), ("G", G), ("Q", Q)):
        if not t.is_cuda or t.dim() != 2 or t.stride(1) != 1:
            raise ValueError(f"{name} must be a 2-D CUDA tensor with unit column stride")
    if X.dtype != torch.float32 or M.dtype != torch.float32 or Q.dtype != torch.float32:
        raise ValueError("X, M and Q must be float32")
    if G.dtype == torch.float32:
        gd = DION_F32
    elif G.dtype == torch.bfloat16:
        gd = DION_BF16
    else:
        raise ValueError("G must be float32 or bfloat16")
    m, n = X.shape
    if tuple(M.shape) != (m, n) or tuple(G.shape) != (m, n) or Q.shape[0] != (m if transposed else n):
        raise ValueError("shape mismatch between X, M, G and Q")
    d = DionMatrix()
    d.m, d.n, d.r = m, n, Q.shape[1]
    d.X, d.ldx = X.data_ptr(), X.stride(0)
    d.M, d.ldm = M.data_ptr(), M.stride(0)
    d.G, d.ldg, d.g_dtype = G.data_ptr(), G.stride(0), gd
    d.Q, d.ldq = Q.data_ptr(), Q.stride(0)
    if colnorm_out is not None:
        if (not colnorm_out.is_cuda or colnorm_out.dtype != torch.float32
                or colnorm_out.numel() < Q.shape[1] or not colnorm_out.is_contiguous()):
            raise ValueError("colnorm_out must be a contiguous float32 CUDA tensor of >= r elements")
        d.colnorm_out = colnorm_out.data_ptr()
    else:
        d.colnorm_out = None
    d.transposed = int(bool(transposed))
    if sketch is not None:
        if (not sketch.is_cuda or sketch.dtype != torch.float32 or sketch.dim() != 2 or sketch.stride(1) != 1
                or sketch.shape[1] != (n if transposed else m)):
            raise ValueError("sketch must be a float32 CUDA matrix with one column per panel row")
        d.sketch, d.sketch_rows, d.ld_sketch = sketch.data_ptr(), sketch.shape[0], sketch.stride(0)
    else:
        d.sketch, d.sketch_rows, d.ld_sketch = None, 0, 0
    return d


def step_noalloc(X, M, G, Q, lr: float, mu: float = 0.95, eps: float = 1e-8, colnorm_out=None,
                 stream=None, transposed: bool = False) -> None:
    """One Dion step through ``dion_step_noalloc``: no context, no device allocation; the
    scratch is the library's built-in 24 MiB array on the current device.  Calls must not
    overlap on the GPU.  Raises DionError(-8) when the shape needs more scratch than that."""
    d = matrix_desc(X, M, G, Q, colnorm_out, transposed)
    _check(load_library().dion_step_noalloc(ctypes.byref(d), float(lr), float(mu), float(eps),
                                            _stream_ptr(stream)))


def noalloc_scratch_limit() -> int:
    return int(load_library().dion_noalloc_scratch_limit())


class Dion:
    """A library context (``dion_init`` .. ``dion_destroy``)."""

    def __init__(self, mu: float = 0.95, eps: float = 1e-8, precision: int = PREC_FP32,
                 orth: int = ORTH_AUTO, engine: int = ENGINE_AUTO, device: Optional[int] = None,
                 workspace_bytes: int = 0):
        lib = load_library()
        if device is None:
            device = torch.cuda.current_device()
        cfg = DionConfig()
        lib.dion_default_config(ctypes.byref(cfg))
        cfg.mu, cfg.eps = mu, eps
        cfg.precision, cfg.orth, cfg.engine = precision, orth, engine
        cfg.device, cfg.workspace_bytes = int(device), int(workspace_bytes)
        self._lib = lib
        self._ctx = ctypes.c_void_p()
        _check(lib.dion_init(ctypes.byref(self._ctx), ctypes.byref(cfg)))
        self.device = int(device)

    def step(self, X, M, G, Q, lr: float, colnorm_out=None, stream=None, transposed: bool = False,
             sketch=None) -> None:
        d = matrix_desc(X, M, G, Q, colnorm_out, transposed, sketch)
        _check(self._lib.dion_step(self._ctx, ctypes.byref(d), float(lr), _stream_ptr(stream)))

    def step_desc(self, desc: DionMatrix, lr: float, stream_ptr: int) -> None:
        """dion_step on a prebuilt descriptor (no per-call marshalling)."""
        _check(self._lib.dion_step(self._ctx, ctypes.byref(desc), float(lr), stream_ptr))

    @staticmethod
    def pack(descs: Sequence[DionMatrix]):
        arr = (DionMatrix * len(descs))(*descs)
        return arr

    def step_grouped(self, mats: Iterable[Tuple], lr: float, stream=None) -> None:
        """mats: iterable of (X, M, G, Q), (X, M, G, Q, colnorm_out) or
        (X, M, G, Q, colnorm_out, transposed[, sketch])."""
        descs: List[DionMatrix] = [matrix_desc(*t) for t in mats]
        arr = self.pack(descs)
        _check(self._lib.dion_step_grouped(self._ctx, arr, len(descs), float(lr), _stream_ptr(stream)))

    def step_grouped_packed(self, arr, count: int, lr: float, stream_ptr: int) -> None:
        _check(self._lib.dion_step_grouped(self._ctx, arr, int(count), float(lr), stream_ptr))

    def lazy_step(self, X, M, G, Q, lr: float, refresh: bool, colnorm_out=None, stream=None) -> None:
        d = matrix_desc(X, M, G, Q, colnorm_out)
        _check(self._lib.dion_lazy_step(self._ctx, ctypes.byref(d), float(lr), int(bool(refresh)),
                                        _stream_ptr(stream)))

    def dp_project(self, desc: DionMatrix, P: torch.Tensor, flag: torch.Tensor, stream=None) -> None:
        """P <- (M + G) Q for the compressed data-parallel sync; the caller then averages P over the ranks."""
        _check(self._lib.dion_dp_project(self._ctx, ctypes.byref(desc), P.data_ptr(), flag.data_ptr(), _stream_ptr(stream)))

    def dp_factor(self, desc: DionMatrix, PU: torch.Tensor, W: torch.Tensor, flag: torch.Tensor, stream=None) -> None:
        """PU: averaged P in, U out; W <- (M + G)^T U; the caller then averages W over the ranks."""
        _check(self._lib.dion_dp_factor(self._ctx, ctypes.byref(desc), PU.data_ptr(), W.data_ptr(), flag.data_ptr(),
                                        _stream_ptr(stream)))

    def dp_finish(self, desc: DionMatrix, U: torch.Tensor, W: torch.Tensor, flag: torch.Tensor, lr: float,
                  stream=None) -> None:
        _check(self._lib.dion_dp_finish(self._ctx, ctypes.byref(desc), U.data_ptr(), W.data_ptr(), flag.data_ptr(),
                                        float(lr), _stream_ptr(stream)))

    # 1D-sharded Dion (Algorithm 3): the per-rank pieces; the caller makes the collectives between them
    def shard_project(self, desc: DionMatrix, n_total: int, P: torch.Tensor, flag: torch.Tensor, stream=None) -> None:
        _check(self._lib.dion_shard_project(self._ctx, ctypes.byref(desc), int(n_total), P.data_ptr(), flag.data_ptr(),
                                            _stream_ptr(stream)))

    def orthonormalize(self, m: int, r: int, n_total: int, PU: torch.Tensor, flag: torch.Tensor, stream=None) -> None:
        _check(self._lib.dion_orthonormalize(self._ctx, int(m), int(r), int(n_total), PU.data_ptr(), flag.data_ptr(),
                                             _stream_ptr(stream)))

    def shard_factor(self, desc: DionMatrix, n_total: int, U: torch.Tensor, W: torch.Tensor, colsumsq: torch.Tensor,
                     flag: torch.Tensor, stream=None) -> None:
        _check(self._lib.dion_shard_factor(self._ctx, ctypes.byref(desc), int(n_total), U.data_ptr(), W.data_ptr(),
                                           colsumsq.data_ptr(), flag.data_ptr(), _stream_ptr(stream)))

    def shard_finish(self, desc: DionMatrix, n_total: int, U: torch.Tensor, W: torch.Tensor, colsumsq: torch.Tensor,
                     flag: torch.Tensor, lr: float, stream=None) -> None:
        _check(self._lib.dion_shard_finish(self._ctx, ctypes.byref(desc), int(n_total), U.data_ptr(), W.data_ptr(),
                                           colsumsq.data_ptr(), flag.data_ptr(), float(lr), _stream_ptr(stream)))

    def lazy_step_desc(self, desc: DionMatrix, lr: float, refresh: bool, stream_ptr: int) -> None:
        _check(self._lib.dion_lazy_step(self._ctx, ctypes.byref(desc), float(lr), int(bool(refresh)), stream_ptr))

    def workspace_bytes(self, m: int, n: int, r: int) -> int:
        return int(self._lib.dion_workspace_bytes(self._ctx, m, n, r))

    def get_status(self, stream=None) -> Tuple[int, int]:
        """Synchronises the stream; returns (status bits, steps skipped) and clears both."""
        st, sk = ctypes.c_int(0), ctypes.c_int(0)
        _check(self._lib.dion_get_status(self._ctx, _stream_ptr(stream), ctypes.byref(st), ctypes.byref(sk)))
        return st.value, sk.value

    def profile_enable(self, on: bool) -> None:
        _check(self._lib.dion_profile_enable(self._ctx, int(bool(on))))

    def profile_read(self):
        """Returns ({phase: ms}, {phase: launches}) summed over the recorded steps."""
        ms = (ctypes.c_float * len(PHASES))()
        nl = (ctypes.c_int64 * len(PHASES))()
        _check(self._lib.dion_profile_read(self._ctx, ms, nl))
        return ({p: float(ms[i]) for i, p in enumerate(PHASES)},
                {p: int(nl[i]) for i, p in enumerate(PHASES)})

    def orth_rounds(self, stream=None) -> int:
        """Adaptive Cholesky QR rounds executed since the last call (synchronises)."""
        n = ctypes.c_int64(0)
        _check(self._lib.dion_get_orth_rounds(self._ctx, _stream_ptr(stream), ctypes.byref(n)))
        return int(n.value)

    def fallbacks(self, stream=None) -> int:
        """Matrices redone by the device-side fallback of CholeskyQR2 since the last call (synchronises)."""
        n = ctypes.c_int64(0)
        _check(self._lib.dion_get_fallbacks(self._ctx, _stream_ptr(stream), ctypes.byref(n)))
        return int(n.value)

    def launch_count(self) -> int:
        return int(self._lib.dion_launch_count(self._ctx))

    def close(self) -> None:
        if self._ctx:
            self._lib.dion_destroy(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

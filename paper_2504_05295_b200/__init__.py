"""B200-native (sm_100a) single-device Dion optimizer step.

The hot path lives in ``csrc/`` (CUDA kernels behind a C-ABI shared library);
``binding`` marshals torch device pointers into it.  ``inputs`` draws the
seeded synthetic workloads.  Nothing here falls back to the CPU.
"""
__all__ = ["inputs"]

// Shared declarations of the Dion CUDA library (device + host helpers).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dion.h"

namespace dion {

typedef int64_t i64;

// How an operand element is formed from memory.
enum : int { ADD_NONE = 0, ADD_F32 = 1, ADD_BF16 = 2 };
// What the epilogue does with an accumulator.
enum : int {
  EPI_STORE = 0,      // C = alpha * acc
  EPI_SUB = 1,        // C = C - alpha * acc
  EPI_ADD2_SUB = 2,   // C = C + C2 - alpha * acc   (error feedback: M <- M + G - beta U R^T)
  EPI_C2_SUB = 3      // C = C2 - alpha * acc       (blocked triangular solve; C2 is fp32)
};
// Which output tiles exist.
enum : int { TRI_FULL = 0, TRI_LOWER = 1 };

// One (optionally batched, optionally split-K) product C = op(A) * op(B).
// A(i,k) = A[i*a_si + k*a_sk] (+ A2(i,k) of dtype a2_mode with its own strides)
// B(k,j) = B[k*b_sk + j*b_sn]
// C(i,j) = C[i*ldc + j]
constexpr int GEMM_TAB_MAX = 64;   // most matrices in one batched tensor-engine launch with per-matrix output pointers

// Per-matrix pointers of a chain for the elementwise kernels that run once over all its matrices.
struct ChainPtrs { const void* p[GEMM_TAB_MAX]; };

struct GemmArgs {
  i64 M, N, K;
  const float* A; i64 a_si, a_sk;
  const void* A2; i64 a2_si, a2_sk; int a2_mode;
  const float* B; i64 b_sk, b_sn;
  float* C; i64 ldc;
  int epi;
  const void* C2; i64 ldc2; int c2_mode;
  float alpha;
  const float* alpha_dev;      // optional: alpha is multiplied by *alpha_dev ...
  i64 alpha_dev_stride;        // ... of entry b of the outer batch: alpha_dev[b * alpha_dev_stride]
  int batch; i64 bsA, bsB, bsC;  // batch count and element strides
  int batch2; i64 bs2;           // outer batch (one per matrix of a grouped call): stride of A, B, C alike
  i64 skip_stride;               // ints between the skip flags of consecutive outer batch entries
  int c2_batched;                // C2 is fp32 and moves with the outer batch too (bs2 elements per entry)
  float* const* c_tab;           // tensor engine, outer batch: HOST arrays of batch2 (<= GEMM_TAB_MAX) pointers, the C (and C2) of
  const void* const* c2_tab;     // every entry (the caller's arrays, at no common stride); copied into the launch parameters
  int splits; float* part;       // split-K: partial sums, [splits][M][N]
  int tri;                       // TRI_LOWER: only the elements on or below the diagonal are needed (tiles above it are skipped)
  int klimit;                    // 1: B(k,j) == 0 for k > j  (K loop ends at the tile's last column)
  const int* skip_flag;          // optional: if *skip_flag != 0 the kernel does nothing
  int precise;                   // tensor engine: keep the small split terms in their own accumulator
  int ab16;                      // tensor engine only: A and B point to bf16 arrays (strides in elements), no addend
  const void* A16lo;             // with ab16: A and B are PAIRS of bf16 arrays, x ~ hi + lo (A, B point to the "hi" arrays, these
  const void* B16lo;             // to the "lo" arrays of the same shape and strides): three bf16 MMAs per K step, ~1e-5 relative
  int f16;                       // with ab16 (no pairs): the arrays hold IEEE half values instead of bf16 (11 significant bits)
  int tf32x1;                    // tensor engine, fp32 mode: the operands' values fit TF32 already (k_round_tf32): one MMA
                                 // per K step instead of the three-term split.  Ignored by the FMA engine.
};

// Programmatic dependent launch (the small kernels of the serial Cholesky chain): lets the next
// launch of the stream be scheduled while this grid runs, then waits until the grids this one
// depends on have completed and their writes are visible.  A kernel launched without the
// attribute passes through both at once.
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ float load_add(const void* p, i64 off, int mode) {
  if (mode == ADD_F32) return reinterpret_cast<const float*>(p)[off];
  if (mode == ADD_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[off]);
  return 0.f;
}

}  // namespace dion

/* Internal test hook of the Dion CUDA library (not part of the public C-ABI):
 * runs one product C = op(A) * op(B) with the fused operand formation and
 * epilogues on a chosen engine, so that the tensor-core kernels can be checked in
 * isolation.  All pointers are DEVICE pointers except `args`. */
#ifndef DION_INTERNAL_H_
#define DION_INTERNAL_H_
#include <stdint.h>
#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int64_t M, N, K;
  const float* A; int64_t a_si, a_sk;            /* A(i,k) = A[i*a_si + k*a_sk]            */
  const void* A2; int64_t a2_si, a2_sk; int a2_mode; /* 0 none, 1 += fp32, 2 += bf16         */
  const float* B; int64_t b_sk, b_sn;            /* B(k,j) = B[k*b_sk + j*b_sn]            */
  float* C; int64_t ldc;
  int epi;                                       /* 0 C=a*acc, 1 C-=a*acc, 2 C=C+C2-a*acc  */
  const void* C2; int64_t ldc2; int c2_mode;
  float alpha;
  int tri;                                       /* 1: only elements on or below the diagonal are guaranteed */
  int klimit;                                    /* 1: B(k,j) = 0 for k > j                */
  int precise;                                   /* 1: split accumulators (tensor engine)  */
  int ab16;                                      /* 1: A and B are bf16 arrays (tensor engine) */
  int tf32x1;                                    /* 1: single-pass TF32 (tensor engine, fp32 mode; operands pre-rounded) */
  int variant;                                   /* tensor engine: bit 0 operands through registers instead of TMA;
                                                    bit 1 (with bit 0) one producer arrival is withheld and every wait
                                                    has a 1 ms budget: the kernel must give up, set DION_STATUS_TIMEOUT
                                                    in *status and return */
  const void* A16lo;                             /* with ab16: the "lo" arrays of bf16 operand pairs (x ~ hi + lo; A, B */
  const void* B16lo;                             /* are the "hi" arrays), or NULL                                        */
  int f16;                                       /* with ab16 (no pairs): the arrays hold IEEE half values */
} dion_debug_gemm_args;

/* engine: 1 = fp32 FMA, 2 = tensor cores (returns DION_ERR_UNSUPPORTED if the
 * product does not qualify).  precision: dion_precision.  part: split-K scratch of
 * part_floats floats (may be NULL).  status: device int receiving DION_STATUS_* bits. */
int dion_debug_gemm(int engine, int precision, const dion_debug_gemm_args* args, float* part,
                    int64_t part_floats, int* status, void* cuda_stream);

/* The estimate of |U1^T U1 - I|_F^2 that the most recent step's CholeskyQR2 check measured (first matrix of
 * its chain); synchronises `cuda_stream`.  `ctx` is a dion_ctx. */
struct dion_ctx;
int dion_debug_orth_measure(struct dion_ctx* ctx, void* cuda_stream, float* estimate);

/* on = 0: the tensor-engine products of a grouped call's chain are launched matrix by matrix instead of once
 * over all matrices of the chain (the results must not depend on it). */
int dion_debug_chain_batch(struct dion_ctx* ctx, int on);

#ifdef __cplusplus
}
#endif
#endif

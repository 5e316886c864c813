// Small kernels of the orthonormalization (r x r factor work) and of ColNorm.
#pragma once

#include "dion_common.cuh"

namespace dion {

constexpr int NB = 64;  // diagonal block of the blocked Cholesky / triangular inverse

// Per-step device state of the orthonormalization (ints, one slot per step).
enum : int {
  OS_FAIL = 0,      // the step must not write X, M, Q (breakdown)
  OS_DONE = 1,      // adaptive rounds: the panel is orthonormal, later rounds are skipped
  OS_GOOD = 2,      // adaptive rounds: the last round saw a well-conditioned panel
  OS_FLOORED = 3,   // pivots raised to the floor in the current round
  OS_MINREL = 4,    // float bits: min over columns of pivot / original diagonal, current round
  OS_ROUNDS = 5,    // rounds that did work
  OS_MAXDEV = 6,    // float bits: the estimate of |U1^T U1 - I|_F^2 of the CholeskyQR2 check
  OS_BARRIER = 7,   // arrival counter of the fallback kernel's grid-wide barriers (zero at the start of a step)
  OS_SLOT_INTS = 8
};

// Round set-up on the r x r Gram matrix G (one block): saves diag(G) to gdiag, writes
// shift = scale * trace(G) (fixed summation order) and resets the round statistics.
// Batched: block b works on the matrix whose scratch starts b * wstride floats further and
// whose state slot is b slots further.
// A trace that is not finite means a NaN or Inf in M, G or Q (every entry of the Gram matrix sums over all
// rows of the panel): the step is cancelled and DION_STATUS_NONFINITE raised.
__global__ void k_round_begin(const float* __restrict__ G, i64 ld, i64 r, float scale,
                              float* __restrict__ gdiag, float* __restrict__ shift,
                              int* __restrict__ os, int adaptive, i64 wstride, int* __restrict__ status) {
  pdl_enter();
  G += (i64)blockIdx.x * wstride; gdiag += (i64)blockIdx.x * wstride; shift += (i64)blockIdx.x * wstride;
  os += (i64)blockIdx.x * OS_SLOT_INTS;
  if (adaptive && os[OS_DONE] != 0) return;
  __shared__ float red[256];
  float s = 0.f;
  for (i64 i = threadIdx.x; i < r; i += blockDim.x) {
    const float v = G[i * ld + i];
    gdiag[i] = v;
    s += v;
  }
  red[threadIdx.x] = s;
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {
    if ((int)threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    *shift = red[0] * scale;
    os[OS_FLOORED] = 0;
    os[OS_MINREL] = 0x7f800000;  // +inf
    if (!(fabsf(red[0]) < __int_as_float(0x7f800000)) && os[OS_FAIL] == 0) {   // (a known failure is not reported twice)
      os[OS_FAIL] = 1;
      atomicOr(status, DION_STATUS_NONFINITE);
    }
  }
}

typedef float (*blk_t)[NB + 1];
typedef float (*half_blk_t)[NB / 2 + 1];

// One doubling level of the triangular inverse inside a 64 x 64 block: for every pair of
// adjacent B x B diagonal blocks, X21 = -X22 (L21 X11).  256 threads, two block-wide barriers.
// SUB: the 256 calling threads are the first eight warps of a larger CTA; they meet at a named barrier of their own.
template <bool SUB>
__device__ __forceinline__ void block_sync() {
  if constexpr (SUB) asm volatile("bar.sync 1, 256;" ::: "memory");
  else __syncthreads();
}

template <int B, bool SUB = false>
__device__ __forceinline__ void trtri_level(blk_t L, blk_t X, half_blk_t T, int tid) {
  constexpr int NPAIRS = NB / (2 * B);
  for (int e = tid; e < NPAIRS * B * B; e += 256) {
    const int pr = e / (B * B), rr = (e / B) % B, cc = e % B, base = pr * 2 * B;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;   // X11 is lower triangular: k >= cc; zeros above are stored
    for (int k = cc & ~3; k < B; k += 4) {
      s0 = fmaf(L[base + B + rr][base + k], X[base + k][base + cc], s0);
      s1 = fmaf(L[base + B + rr][base + k + 1], X[base + k + 1][base + cc], s1);
      s2 = fmaf(L[base + B + rr][base + k + 2], X[base + k + 2][base + cc], s2);
      s3 = fmaf(L[base + B + rr][base + k + 3], X[base + k + 3][base + cc], s3);
    }
    T[pr * B + rr][cc] = (s0 + s1) + (s2 + s3);
  }
  block_sync<SUB>();
  for (int e = tid; e < NPAIRS * B * B; e += 256) {
    const int pr = e / (B * B), rr = (e / B) % B, cc = e % B, base = pr * 2 * B;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;   // X22 is lower triangular: k <= rr; zeros above are stored
    for (int k = 0; k <= rr; k += 4) {
      s0 = fmaf(X[base + B + rr][base + B + k], T[pr * B + k][cc], s0);
      s1 = fmaf(X[base + B + rr][base + B + k + 1], T[pr * B + k + 1][cc], s1);
      s2 = fmaf(X[base + B + rr][base + B + k + 2], T[pr * B + k + 2][cc], s2);
      s3 = fmaf(X[base + B + rr][base + B + k + 3], T[pr * B + k + 3][cc], s3);
    }
    X[base + B + rr][base + cc] = -((s0 + s1) + (s2 + s3));
  }
  block_sync<SUB>();
}

// Inverse X of the lower-triangular 64 x 64 block L (shared memory; rdiag[i] = 1 / L[i][i];
// X zero on entry): 16 x 16 diagonal inverses by forward substitution, then doubling.
// Called by all 256 threads after a block-wide barrier; ends with one.
template <bool SUB = false>
__device__ __forceinline__ void invert_block(blk_t L, blk_t X, half_blk_t T, const float* rdiag, int tid) {
  constexpr int W = 16;
  if (tid < NB) {
    const int b0 = (tid / W) * W, q = tid % W;
    float x[W];
#pragma unroll
    for (int i = 0; i < W; ++i) {
      float sacc = (i == q) ? 1.f : 0.f;
#pragma unroll
      for (int k = 0; k < i; ++k)
        if (k >= q) sacc = fmaf(-L[b0 + i][b0 + k], x[k], sacc);
      x[i] = (i >= q) ? sacc * rdiag[b0 + i] : 0.f;
    }
#pragma unroll
    for (int i = 0; i < W; ++i) X[b0 + i][b0 + q] = x[i];
  }
  block_sync<SUB>();
  // ... then [[X11, 0], [-X22 L21 X11, X22]] for block sizes 16 and 32
  trtri_level<16, SUB>(L, X, T, tid);
  trtri_level<32, SUB>(L, X, T, tid);
}

// Cholesky factor and its inverse of the 64 x 64 block held in L (shared memory; lower
// triangle, identity padding beyond a ragged block of jb columns), by the 256 threads of
// a CTA.  On return L holds the factor, X its inverse, deflated[] the deflated columns.
// X must be zero on entry, gd[] hold the floors' reference values, deflated[] zeros,
// and a block-wide barrier must separate those writes from the call.
// The block is factored in four 16-column sub-panels: the 16 x 16 diagonal piece by
// one warp (rows in registers, shuffles, no barrier), the rows below it by one thread per
// row, the trailing update by all threads -- three block-wide barriers per sub-panel
// instead of three per column.  The inverse is built from 16 x 16 inverses by doubling.
template <bool SUB = false>
__device__ __forceinline__ void potrf_block(blk_t L, blk_t X, half_blk_t T, const float* gd, float* rdiag,
                                            int* deflated, int jb, float floor_rel, int* __restrict__ os,
                                            int* __restrict__ status) {
  constexpr int W = 16;    // base blocks of the inverse
  constexpr int WF = 8;    // sub-panel width of the factorization
  const int tid = threadIdx.x;
  int floored = 0, failed = 0;
  float minrel = __int_as_float(0x7f800000);
  const float inf = __int_as_float(0x7f800000);
#pragma unroll 1
  for (int c0 = 0; c0 < NB; c0 += WF) {
    if (tid == 0) {
      // WF x WF diagonal piece: one thread, the lower triangle in registers.  The chain
      // pivot -> rsqrt -> scale -> update of the next pivot is serial whatever the thread
      // count; one thread runs it without any barrier or shuffle.  Padding columns of a
      // ragged block (unit diagonal, gd = 0) pass every test.
      float a[WF][WF], g[WF];
#pragma unroll
      for (int i = 0; i < WF; ++i) {
        g[i] = gd[c0 + i];
#pragma unroll
        for (int c = 0; c <= i; ++c) a[i][c] = L[c0 + i][c0 + c];
      }
#pragma unroll
      for (int j = 0; j < WF; ++j) {
        float p = a[j][j];
        const float fl = floor_rel * g[j];           // 0 in the plain mode
        bool defl = false;
        if (!(p > fl) || !(p < inf)) {
          if (floor_rel > 0.f) {
            p = (fl > 0.f && fl < inf) ? fl : 1.f;   // zero or non-finite column: unit pivot
            defl = true;
            ++floored;
          } else {
            failed = 1;
            p = 1.f;
          }
        } else {
          minrel = fminf(minrel, __fdividef(p, g[j]));
        }
        const float inv = rsqrtf(p);
        const float sc = defl ? 0.f : inv;
        a[j][j] = p * inv;
        rdiag[c0 + j] = inv;
        if (defl) deflated[c0 + j] = 1;
#pragma unroll
        for (int i = j + 1; i < WF; ++i) a[i][j] *= sc;
#pragma unroll
        for (int c = j + 1; c < WF; ++c)
#pragma unroll
          for (int i = c; i < WF; ++i) a[i][c] = fmaf(-a[i][j], a[c][j], a[i][c]);
      }
#pragma unroll
      for (int i = 0; i < WF; ++i)
#pragma unroll
        for (int c = 0; c <= i; ++c) L[c0 + i][c0 + c] = a[i][c];
    }
    else if (tid >= 32 && c0 > 0) {
      // meanwhile warps 1-7 finish the trailing update of the previous sub-panel: its columns from
      // c0 + WF on (the WF columns the piece and the next panel need were updated right away)
      const int p0 = c0 - WF;                       // the previous sub-panel's first column
      const int t2 = tid - 32, ty = t2 >> 4, tx = t2 & 15;
      for (int i = c0 + WF + ty; i < NB; i += 14)
        for (int c = c0 + WF + tx; c <= i; c += 16) {
          float sacc = 0.f;
#pragma unroll
          for (int k = 0; k < WF; ++k) sacc = fmaf(L[i][p0 + k], L[c][p0 + k], sacc);
          L[i][c] -= sacc;
        }
    }
    block_sync<SUB>();
    const int below = NB - c0 - WF;   // rows under the diagonal piece
    if (tid < below) {
      const int i = c0 + WF + tid;
      float x[WF];
#pragma unroll
      for (int j = 0; j < WF; ++j) {
        float sacc = L[i][c0 + j];
#pragma unroll
        for (int k = 0; k < j; ++k) sacc = fmaf(-x[k], L[c0 + j][c0 + k], sacc);
        x[j] = deflated[c0 + j] ? 0.f : sacc * rdiag[c0 + j];
      }
#pragma unroll
      for (int j = 0; j < WF; ++j) L[i][c0 + j] = x[j];
    }
    block_sync<SUB>();
    // trailing update, first part: the WF columns that the next diagonal piece and the panel below
    // it need (thread -> (row, column)); the rest is deferred to run beside the next diagonal piece
    for (int e = tid; e < below * WF; e += 256) {
      const int i = c0 + WF + e / WF, c = c0 + WF + e % WF;
      if (c <= i) {
        float sacc = 0.f;
#pragma unroll
        for (int k = 0; k < WF; ++k) sacc = fmaf(L[i][c0 + k], L[c][c0 + k], sacc);
        L[i][c] -= sacc;
      }
    }
    block_sync<SUB>();
  }
  if (tid == 0) {
    if (floor_rel > 0.f) {
      if (floored) atomicAdd(&os[OS_FLOORED], floored);
      atomicMin(&os[OS_MINREL], __float_as_int(minrel));
    } else if (failed) {
      os[OS_FAIL] = 1;
      if (status != nullptr) atomicOr(status, DION_STATUS_BREAKDOWN);   // nullptr: a fallback follows in the same step
    }
  }

  invert_block<SUB>(L, X, T, rdiag, tid);
}

// Cholesky of one jb x jb (jb <= 64) diagonal block, in place (lower factor, the
// strict upper part of the block is zeroed), plus the inverse of that factor into
// Dinv (64 x 64, row-major, zero padded).
// floor_rel == 0 (plain Cholesky QR): a pivot that is <= 0 or not finite sets
//   os[OS_FAIL] and the BREAKDOWN status bit and is replaced by 1 so that everything
//   downstream stays finite.
// floor_rel > 0 (adaptive rounds): a pivot below floor_rel * gdiag[j] (gdiag = the
//   diagonal of the Gram matrix before elimination) is below the rounding noise of
//   the Gram matrix.  Column j is then deflated: its diagonal entry becomes
//   sqrt(floor), the entries below it zero, so the noisy column never reaches the
//   trailing matrix.  The factor stays triangular and nonsingular for any panel;
//   the round only improves the conditioning and a later round finishes the job.
//   DinvP is Dinv with the rows of deflated columns zeroed: the panel below this
//   block is multiplied by DinvP^T, which yields the zero columns of the factor.
__global__ void __launch_bounds__(256) k_potrf_diag(float* __restrict__ A, i64 ld, int jb,
                                                    float* __restrict__ Dinv, float* __restrict__ DinvP,
                                                    const float* __restrict__ gdiag, float floor_rel,
                                                    int* __restrict__ os, int adaptive,
                                                    int* __restrict__ status, i64 wstride) {
  {  // batched: block b -> matrix b
    const i64 wo = (i64)blockIdx.x * wstride;
    A += wo; Dinv += wo; DinvP += wo; gdiag += wo;
    os += (i64)blockIdx.x * OS_SLOT_INTS;
  }
  pdl_enter();
  if (adaptive && os[OS_DONE] != 0) return;
  __shared__ float L[NB][NB + 1];
  __shared__ float X[NB][NB + 1];
  __shared__ float T[NB / 2][NB / 2 + 1];
  __shared__ float gd[NB];
  __shared__ float rdiag[NB];     // 1 / L[j][j]
  __shared__ int deflated[NB];
  const int tid = threadIdx.x;
  if (tid < NB) {
    deflated[tid] = 0;
    gd[tid] = (floor_rel > 0.f && tid < jb) ? gdiag[tid] : 0.f;
  }
  {
    float v[NB * NB / 256];
#pragma unroll
    for (int l = 0; l < NB * NB / 256; ++l) {
      const int e = tid + l * 256, i = e / NB, c = e % NB;
      v[l] = (i < jb && c <= i) ? A[(i64)i * ld + c] : 0.f;
    }
#pragma unroll
    for (int l = 0; l < NB * NB / 256; ++l) {
      const int e = tid + l * 256, i = e / NB, c = e % NB;
      float x = v[l];
      if (i == c && i >= jb) x = 1.f;   // identity padding of a ragged last block
      L[i][c] = x;
      X[i][c] = 0.f;
    }
  }
  __syncthreads();

  potrf_block(L, X, T, gd, rdiag, deflated, jb, floor_rel, os, status);
  for (int e = tid; e < NB * NB; e += 256) {
    const int i = e / NB, c = e % NB;
    if (i < jb && c < jb) A[(i64)i * ld + c] = (c <= i) ? L[i][c] : 0.f;
    Dinv[e] = X[i][c];
    DinvP[e] = deflated[i] ? 0.f : X[i][c];
  }
}

// CholeskyQR2 of a small panel (rows x r, r <= 64, rows <= TINY_MAX_ROWS, leading dimension r) in ONE launch, one
// CTA of 1024 threads per matrix, the panel resident in shared memory: Gram matrix (3xTF32 on the warp-level tensor
// path), Cholesky factor and its inverse (potrf_block, on the first eight warps), U1 = P L^-T (3xTF32), then the second round's Gram matrix G2 = U1^T U1, which
// also says exactly how far U1 is from orthonormal: |G2 - I|_F^2 <= tau_f^2 r -> done after one round (the same
// test the probe of the large panels estimates), else the second round runs on G2.  Replaces some seventeen
// launches of a step on such a panel.  Every sum has a fixed order: same bits on every run.
// State as the launch chain leaves it: OS_MAXDEV (the deviation), OS_DONE = 1, OS_ROUNDS and *rounds_total (1 or
// 2); a pivot that is not positive raises OS_FAIL (and DION_STATUS_BREAKDOWN unless `status_fail` is nullptr: a
// fallback follows), the panel is then left to the fallback; a Gram trace that is not finite raises OS_FAIL and
// DION_STATUS_NONFINITE.  Pin may equal Pout.
constexpr int TINY_MAX_ROWS = 512;
constexpr int TINY_THREADS = 1024;
// Row strides (floats) that keep the fragment loads of the two products off each other's banks: a lane reads
// (row ft, column fg) of the panel for the Gram matrix (stride = 8 mod 32: no conflict) and (row fg, column ft)
// of it (two-way) and of the inverse (copied to stride = 4 mod 32: none) for U.
constexpr int TINY_LD = NB + 8;
constexpr int TINY_XLD = NB + 4;
constexpr int TINY_BLK = NB * (NB + 1);     // floats of a 64 x 65 block
inline int tiny_rows_pad(i64 rows) { return (int)((rows + 15) / 16 * 16); }
inline int tiny_cholqr2_smem(i64 rows) {    // panel (rows padded to 16), L, X, the copy of X, T, gd, rdiag, red, deflated
  return (int)sizeof(float) * (tiny_rows_pad(rows) * TINY_LD + 2 * TINY_BLK + NB * TINY_XLD + (NB / 2) * (NB / 2 + 1) + 2 * NB + TINY_THREADS) +
         (int)sizeof(int) * NB;
}

// The two small products of the kernel run on the warp-level tensor-core path (m16n8k8, TF32 operands, fp32
// accumulation) as 3xTF32: x = hi + lo with hi = x truncated to TF32; lo x hi + hi x lo first, hi x hi last.
__device__ __forceinline__ void mma_tf32_16x8x8(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo) {
  hi = __float_as_uint(x) & 0xffffe000u;
  lo = __float_as_uint(x - __uint_as_float(hi));
}
template <int NA, int NB_>
__device__ __forceinline__ void mma_3xtf32(float (&c)[4], const float (&a)[NA], const float (&b)[NB_]) {
  static_assert(NA == 4 && NB_ == 2, "m16n8k8 fragments");
  uint32_t ah[4], al[4], bh[2], bl[2];
#pragma unroll
  for (int x = 0; x < 4; ++x) split_tf32(a[x], ah[x], al[x]);
#pragma unroll
  for (int x = 0; x < 2; ++x) split_tf32(b[x], bh[x], bl[x]);
  mma_tf32_16x8x8(c, al, bh);
  mma_tf32_16x8x8(c, ah, bl);
  mma_tf32_16x8x8(c, ah, bh);
}

__global__ void __launch_bounds__(TINY_THREADS) k_tiny_cholqr2(const float* __restrict__ Pin, float* __restrict__ Pout, int rows, int r,
                                                               int* __restrict__ os, float tau_f, int* __restrict__ rounds_total,
                                                               int* __restrict__ status_fail, int* __restrict__ status_always,
                                                               i64 wstride) {
  Pin += (i64)blockIdx.x * wstride; Pout += (i64)blockIdx.x * wstride;
  os += (i64)blockIdx.x * OS_SLOT_INTS;
  pdl_enter();
  extern __shared__ __align__(16) float tiny_smem[];
  const int rows_pad = (rows + 15) / 16 * 16;
  float* Ps = tiny_smem;                                              // rows_pad x TINY_LD; rows beyond `rows` and columns beyond r are zero
  float* blocks = Ps + rows_pad * TINY_LD;
  blk_t L = reinterpret_cast<blk_t>(blocks);
  blk_t X = reinterpret_cast<blk_t>(blocks + TINY_BLK);
  float* XS = blocks + 2 * TINY_BLK;                                  // the inverse, row stride TINY_XLD
  half_blk_t T = reinterpret_cast<half_blk_t>(XS + NB * TINY_XLD);
  float* gd = XS + NB * TINY_XLD + (NB / 2) * (NB / 2 + 1);
  float* rdiag = gd + NB;
  float* red = rdiag + NB;                                            // TINY_THREADS
  int* deflated = reinterpret_cast<int*>(red + TINY_THREADS);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int fg = lane >> 2, ft = lane & 3;                            // fragment coordinates of the lane

  if (r % 4 == 0 && (reinterpret_cast<uintptr_t>(Pin) & 15u) == 0) {
    // four 16-byte loads in flight per thread
    const int nv = rows * r / 4;
    const float4* src = reinterpret_cast<const float4*>(Pin);
    for (int base = 0; base < nv; base += TINY_THREADS * 4) {
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int idx = base + u * TINY_THREADS + tid;
        v[u] = (idx < nv) ? __ldg(src + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int idx = base + u * TINY_THREADS + tid;
        if (idx < nv) {
          float* d = Ps + (4 * idx / r) * TINY_LD + (4 * idx % r);
          d[0] = v[u].x; d[1] = v[u].y; d[2] = v[u].z; d[3] = v[u].w;
        }
      }
    }
    if (r < NB)
      for (int e = tid; e < rows * (NB - r); e += TINY_THREADS) Ps[(e / (NB - r)) * TINY_LD + r + e % (NB - r)] = 0.f;
  } else {
#pragma unroll 4
    for (int e = tid; e < rows * NB; e += TINY_THREADS) {
      const int i = e / NB, c = e % NB;
      Ps[i * TINY_LD + c] = (c < r) ? Pin[(i64)i * r + c] : 0.f;
    }
  }
  for (int e = rows * NB + tid; e < rows_pad * NB; e += TINY_THREADS) Ps[(e / NB) * TINY_LD + e % NB] = 0.f;
  __syncthreads();

  // G = P^T P (64 x 64, K = rows_pad): warp w owns the 16 x 8 tile (w / 8, w % 8); lane (fg, ft) then holds
  // G[m0 + fg][n0 + 2 ft], [..][n0 + 2 ft + 1], G[m0 + fg + 8][n0 + 2 ft], [..][n0 + 2 ft + 1].
  const int m0 = (warp >> 3) * 16, n0 = (warp & 7) * 8;
  float acc[4];
  auto gram = [&]() {
    acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
#pragma unroll 4
    for (int k0 = 0; k0 < rows_pad; k0 += 8) {
      const float* r0 = Ps + (k0 + ft) * TINY_LD;
      const float* r1 = Ps + (k0 + ft + 4) * TINY_LD;
      const float a[4] = {r0[m0 + fg], r0[m0 + fg + 8], r1[m0 + fg], r1[m0 + fg + 8]};    // A(m, k) = P[k][m]
      const float b[2] = {r0[n0 + fg], r1[n0 + fg]};                                      // B(k, n) = P[k][n]
      mma_3xtf32(acc, a, b);
    }
  };
  // the Gram matrix from the registers into L: lower triangle, zero above, identity beyond column r; X, gd,
  // deflated reset
  auto stage_factor_input = [&]() {
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const int i = m0 + fg + ((x & 2) ? 8 : 0), c = n0 + 2 * ft + (x & 1);
      float v = (i < r && c <= i) ? acc[x] : 0.f;
      if (i == c && i >= r) v = 1.f;
      L[i][c] = v;
      X[i][c] = 0.f;
      if (i == c) red[i] = (i < r) ? acc[x] : 0.f;      // the diagonal, for the trace
    }
    if (tid < NB) { deflated[tid] = 0; gd[tid] = 0.f; }
  };
  // U = P X^T in place (X lower triangular, its zeros above the diagonal stored): work item = 16 rows x 32
  // columns, K = 64; the items of a sweep are all computed before any entry of the panel is overwritten.
  auto apply_inverse = [&]() {
    for (int e = tid; e < NB * NB; e += TINY_THREADS) XS[(e / NB) * TINY_XLD + e % NB] = X[e / NB][e % NB];
    __syncthreads();
    const int items = (rows_pad / 16) * 2;
    for (int it0 = 0; it0 < items; it0 += TINY_THREADS / 32) {
      const int it = it0 + warp;
      const int i0 = (it >> 1) * 16, c0 = (it & 1) * 32;
      float y[4][4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) y[nt][0] = y[nt][1] = y[nt][2] = y[nt][3] = 0.f;
      if (it < items) {
#pragma unroll 2
        for (int k0 = 0; k0 < NB; k0 += 8) {
          const float* r0 = Ps + (i0 + fg) * TINY_LD + k0;
          const float* r1 = Ps + (i0 + fg + 8) * TINY_LD + k0;
          const float a[4] = {r0[ft], r1[ft], r0[ft + 4], r1[ft + 4]};                    // A(m, k) = P[i0 + m][k]
#pragma unroll
          for (int nt = 0; nt < 4; ++nt) {
            const float* xr = XS + (c0 + 8 * nt + fg) * TINY_XLD + k0;
            const float b[2] = {xr[ft], xr[ft + 4]};                                      // B(k, n) = X[n][k]
            mma_3xtf32(y[nt], a, b);
          }
        }
      }
      __syncthreads();
      if (it < items) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          const int c = c0 + 8 * nt + 2 * ft;
          float* w0 = Ps + (i0 + fg) * TINY_LD + c;
          float* w1 = Ps + (i0 + fg + 8) * TINY_LD + c;
          w0[0] = y[nt][0]; w0[1] = y[nt][1]; w1[0] = y[nt][2]; w1[1] = y[nt][3];
        }
      }
    }
    __syncthreads();
  };

  gram();
  stage_factor_input();
  __syncthreads();
  if (warp == 8) {      // (a warp that has no part in the factorization: the trace from the staged diagonal, fixed order)
    float tr = red[lane] + red[lane + 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tr += __shfl_xor_sync(0xffffffffu, tr, o);
    if (lane == 0 && !(fabsf(tr) < __int_as_float(0x7f800000)) && os[OS_FAIL] == 0) {
      os[OS_FAIL] = 1;
      atomicOr(status_always, DION_STATUS_NONFINITE);
    }
  }
  if (tid < 256) potrf_block<true>(L, X, T, gd, rdiag, deflated, r, 0.f, os, status_fail);   // (ends with its own barrier)
  __syncthreads();
  const bool failed1 = reinterpret_cast<volatile int*>(os)[OS_FAIL] != 0;   // (written by this CTA's thread 0 before that barrier, or before this launch)
  apply_inverse();

  // the second round's Gram matrix, and with it the first round's distance from orthonormal
  gram();
  float e = 0.f;
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int i = m0 + fg + ((x & 2) ? 8 : 0), c = n0 + 2 * ft + (x & 1);
    if (i < r && c < r) { const float d = acc[x] - ((i == c) ? 1.f : 0.f); e = fmaf(d, d, e); }
  }
  red[tid] = e;
  __syncthreads();
  for (int w = TINY_THREADS / 2; w > 0; w >>= 1) {
    if (tid < w) red[tid] += red[tid + w];
    __syncthreads();
  }
  const float est = red[0];
  const bool done = !failed1 && (est <= tau_f * tau_f * (float)r);      // false for NaN
  if (!done && !failed1) {
    __syncthreads();                 // everyone has read red[0]
    stage_factor_input();
    __syncthreads();
    if (tid < 256) potrf_block<true>(L, X, T, gd, rdiag, deflated, r, 0.f, os, status_fail);
    __syncthreads();
    apply_inverse();
  }
  if (tid == 0) {
    os[OS_MAXDEV] = __float_as_int(est);
    os[OS_DONE] = 1;
    os[OS_ROUNDS] = done ? 1 : 2;
    atomicAdd(rounds_total, done ? 1 : 2);
  }
#pragma unroll 4
  for (int e2 = tid; e2 < rows * r; e2 += TINY_THREADS) {
    const int i = e2 / r, c = e2 % r;
    Pout[(i64)i * r + c] = Ps[i * TINY_LD + c];
  }
}

// Operand tiles of the 64 x 64 x 64 products: rows of 68 floats (16-byte aligned rows for
// 128-bit loads along k; the row patterns below stay free of bank conflicts).
constexpr int MMS = NB + 4;
typedef float (*mm_t)[MMS];

// acc[a][b] += sum_k A[4 ty + a][k] * B[tx + 16 b][k]  (64 x 64 x 64, operands in shared memory)
__device__ __forceinline__ void mm_nt_64(mm_t A, mm_t B, int ty, int tx, float (&acc)[4][4]) {
#pragma unroll 4
  for (int k = 0; k < NB; k += 4) {
    float4 av[4], bv[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) av[a] = *reinterpret_cast<const float4*>(&A[ty * 4 + a][k]);
#pragma unroll
    for (int b = 0; b < 4; ++b) bv[b] = *reinterpret_cast<const float4*>(&B[tx + 16 * b][k]);
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        float t = acc[a][b];
        t = fmaf(av[a].x, bv[b].x, t);
        t = fmaf(av[a].y, bv[b].y, t);
        t = fmaf(av[a].z, bv[b].z, t);
        t = fmaf(av[a].w, bv[b].w, t);
        acc[a][b] = t;
      }
  }
}

constexpr int CHOL_STEP_SMEM = 3 * NB * MMS * (int)sizeof(float);

// The inverse X of the factor of the diagonal square [o, o+sz), 64 x 64 blocks:
//   X_im = -Dinv_i * S_im,   S_im = sum_{k=m}^{i-1} L_ik X_km,   X_mm = Dinv_m   (m < i).
// The sums are accumulated right-looking, one term per launch: as soon as block column kk of the factor
// and block row kk of X are final, every later row adds its term k = kk,
//   S_im (+)= L_{i,kk} X_{kk,m}   (the first term, m = kk, takes X_kk,kk = Dinv_kk),
// and the row that is complete with it (i = kk + 1, `finish`) is multiplied by -Dinv_i.  S_im lives in
// X_im's place in Linv until then.  L is read from Lsrc (the panels the steps have written).  One CTA of
// 256 threads per block and launch: one 64^3 product, two for the finishing row; smem holds two tiles.
__device__ __forceinline__ void inv_term(const float* __restrict__ Lsrc, float* __restrict__ Linv, i64 ld,
                                         const float* __restrict__ Dinv, i64 o, i64 sz, int i, int m, int kk,
                                         bool finish, float* smem) {
  mm_t S0 = reinterpret_cast<mm_t>(smem);
  mm_t S1 = reinterpret_cast<mm_t>(smem + NB * MMS);
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const i64 ri = o + (i64)i * NB, cm = o + (i64)m * NB, rk = o + (i64)kk * NB;
  const int rows_i = (int)((o + sz - ri < NB) ? (o + sz - ri) : NB);
  const bool first = (m == kk);
  const float* Dk = Dinv + (rk / NB) * (NB * NB);
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b)
      acc[a][b] = (!first && ty * 4 + a < rows_i) ? Linv[(ri + ty * 4 + a) * ld + cm + tx + 16 * b] : 0.f;
#pragma unroll 4
  for (int l = 0; l < NB * NB / 256; ++l) {
    const int e = tid + l * 256, rr = e / NB, cc = e % NB;
    S0[rr][cc] = (rr < rows_i) ? Lsrc[(ri + rr) * ld + rk + cc] : 0.f;
    S1[cc][rr] = first ? Dk[e] : Linv[(rk + rr) * ld + cm + cc];   // transposed: the product below is A * B^T
  }
  __syncthreads();
  mm_nt_64(S0, S1, ty, tx, acc);
  if (!finish) {
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b)
        if (ty * 4 + a < rows_i) Linv[(ri + ty * 4 + a) * ld + cm + tx + 16 * b] = acc[a][b];
    return;
  }
  __syncthreads();
  const float* Di = Dinv + (ri / NB) * (NB * NB);
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) S1[tx + 16 * b][ty * 4 + a] = acc[a][b];
#pragma unroll 4
  for (int l = 0; l < NB * NB / 256; ++l) {
    const int e = tid + l * 256;
    S0[e / NB][e % NB] = Di[e];
  }
  __syncthreads();
  float x[4][4] = {};
  mm_nt_64(S0, S1, ty, tx, x);
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b)
      if (ty * 4 + a < rows_i) Linv[(ri + ty * 4 + a) * ld + cm + tx + 16 * b] = -x[a][b];
}

// One step of the right-looking 64-column Cholesky inside the diagonal square [o, o+sz)
// of the Gram matrix, in ONE launch: with the diagonal block of block column j already
// factored (its inverse in DinvP), CTA (bi, bk), bk <= bi, forms the two 64-row pieces
// L_i = A[i][j] DinvP^T and L_k of block column j of the factor, and subtracts
// L_i L_k^T from the trailing block (i, k).  The CTA of the next diagonal block
// (bi = bk = 0) then factors and inverts that block right away, so that the next step
// can start at the next launch; the other CTAs run beside it.  The L pieces go to Lout
// (same offsets as in A): block column j of A is still read by the other CTAs of this
// launch, so it cannot be overwritten here; the caller copies Lout back after the last step.
__global__ void __launch_bounds__(256) k_chol_step(float* __restrict__ A, i64 ld, i64 o, i64 sz, int j,
                                                   float* __restrict__ Dinv, float* __restrict__ DinvP,
                                                   float* __restrict__ Lout, float* __restrict__ Linv,
                                                   const float* __restrict__ gdiag, float floor_rel,
                                                   int* __restrict__ os, int adaptive,
                                                   int* __restrict__ status, i64 wstride) {
  {
    const i64 wo = (i64)blockIdx.y * wstride;
    A += wo; Dinv += wo; DinvP += wo; Lout += wo; Linv += wo; gdiag += wo;
    os += (i64)blockIdx.y * OS_SLOT_INTS;
  }
  // Launched with programmatic stream serialization: the next step's CTAs may be scheduled while
  // this grid still runs (they wait here), which takes the launch latency off the serial chain.
  pdl_enter();
  if (adaptive && os[OS_DONE] != 0) return;
  extern __shared__ __align__(16) float chol_smem[];
  {
    // the CTAs behind the trailing blocks: block column j - 1 of the factor and block row j - 1 of the
    // square's inverse are final since the last launch; every row i >= j of the inverse adds that term
    // (j blocks per row), and row j is complete with it
    const int nblk = (int)((sz + NB - 1) / NB);
    const int nt = nblk - 1 - j;
    const int ntri = nt * (nt + 1) / 2;
    if ((int)blockIdx.x >= ntri) {
      const int x = (int)blockIdx.x - ntri;
      const int i = j + x / j, m = x % j;
      inv_term(Lout, Linv, ld, Dinv, o, sz, i, m, j - 1, i == j, chol_smem);
      return;
    }
  }
  mm_t S0 = reinterpret_cast<mm_t>(chol_smem);
  mm_t S1 = reinterpret_cast<mm_t>(chol_smem + NB * MMS);
  mm_t S2 = reinterpret_cast<mm_t>(chol_smem + 2 * NB * MMS);
  __shared__ float gd[NB];
  __shared__ float rdiag[NB];
  __shared__ int deflated[NB];
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  int bi = 0;
  while ((bi + 1) * (bi + 2) / 2 <= (int)blockIdx.x) ++bi;
  const int bk = (int)blockIdx.x - bi * (bi + 1) / 2;
  const i64 cj = o + (i64)j * NB;                    // first column of block column j
  const i64 ri = cj + (i64)NB * (1 + bi), rk = cj + (i64)NB * (1 + bk);
  const int rows_i = (int)((o + sz - ri < NB) ? (o + sz - ri) : NB);
  const int rows_k = (int)((o + sz - rk < NB) ? (o + sz - rk) : NB);
  const bool diag = (bi == bk);
  const bool next_diag = (bi == 0 && bk == 0);
  const float* DPj = DinvP + (cj / NB) * (NB * NB);
  float cblk[4][4];      // this thread's entries of trailing block (i, k), fetched ahead of the products
  {
    float vi[NB * NB / 256], vk[NB * NB / 256], vd[NB * NB / 256];
#pragma unroll
    for (int l = 0; l < NB * NB / 256; ++l) {
      const int e = tid + l * 256, i = e / NB, c = e % NB;
      vi[l] = (i < rows_i) ? A[(ri + i) * ld + cj + c] : 0.f;
      vk[l] = (!diag && i < rows_k) ? A[(rk + i) * ld + cj + c] : 0.f;
      vd[l] = DPj[e];
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int i = ty * 4 + a, c = tx + 16 * b;
        cblk[a][b] = (i < rows_i && c < rows_k) ? A[(ri + i) * ld + rk + c] : 0.f;
      }
#pragma unroll
    for (int l = 0; l < NB * NB / 256; ++l) {
      const int e = tid + l * 256, i = e / NB, c = e % NB;
      S0[i][c] = vi[l];
      S1[i][c] = vk[l];
      S2[i][c] = vd[l];
    }
  }
  __syncthreads();
  float li[4][4] = {}, lk[4][4] = {};
  mm_nt_64(S0, S2, ty, tx, li);
  if (!diag) mm_nt_64(S1, S2, ty, tx, lk);
  __syncthreads();
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      S0[ty * 4 + a][tx + 16 * b] = li[a][b];
      if (!diag) S1[ty * 4 + a][tx + 16 * b] = lk[a][b];
      if (bk == 0 && ty * 4 + a < rows_i) Lout[(ri + ty * 4 + a) * ld + cj + tx + 16 * b] = li[a][b];
    }
  __syncthreads();
  float acc[4][4] = {};
  mm_nt_64(S0, diag ? S0 : S1, ty, tx, acc);
  if (!next_diag) {
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int i = ty * 4 + a, c = tx + 16 * b;
        if (i < rows_i && c < rows_k) A[(ri + i) * ld + rk + c] = cblk[a][b] - acc[a][b];
      }
    return;
  }
  // the next diagonal block: factor and invert it here.  The three buffers are reused as the
  // factor L (65-float rows, S2: the inverse of the previous block is no longer needed), its
  // inverse X (S1) and the scratch T of the inverse levels (S0).
  blk_t Lb = reinterpret_cast<blk_t>(chol_smem + 2 * NB * MMS);
  blk_t Xb = reinterpret_cast<blk_t>(chol_smem + NB * MMS);
  if (tid < NB) {
    deflated[tid] = 0;
    gd[tid] = (floor_rel > 0.f && tid < rows_i) ? gdiag[ri + tid] : 0.f;
  }
  __syncthreads();                // every thread is done reading S0 / S1 / S2
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int i = ty * 4 + a, c = tx + 16 * b;
      const float v = cblk[a][b] - acc[a][b];
      Lb[i][c] = (c < i) ? v : ((c == i) ? ((i < rows_i) ? v : 1.f) : 0.f);
    }
  for (int e = tid; e < NB * NB; e += 256) Xb[e / NB][e % NB] = 0.f;
  __syncthreads();
  potrf_block(Lb, Xb, reinterpret_cast<half_blk_t>(chol_smem), gd, rdiag, deflated, rows_i, floor_rel, os, status);
  float* Dn = Dinv + (ri / NB) * (NB * NB);
  float* DPn = DinvP + (ri / NB) * (NB * NB);
  for (int e = tid; e < NB * NB; e += 256) {
    const int i = e / NB, c = e % NB;
    if (i < rows_i && c < rows_i) A[(ri + i) * ld + ri + c] = (c <= i) ? Lb[i][c] : 0.f;
    Dn[e] = Xb[i][c];
    DPn[e] = deflated[i] ? 0.f : Xb[i][c];
  }
}

// After the last k_chol_step of a square [o, o+sz): the first CTAs complete the last block row of the
// inverse of the factor (inv_term); the others move the factor's blocks below the block diagonal from
// Lout into A, put the diagonal inverses into Linv and clear Linv above the block diagonal.
constexpr int INV_FINISH_SMEM = 2 * NB * MMS * (int)sizeof(float);
__global__ void __launch_bounds__(256) k_inv_finish(const float* __restrict__ Lout, float* __restrict__ A,
                                                    float* __restrict__ Linv, i64 ld, i64 o, i64 sz,
                                                    const float* __restrict__ Dinv,
                                                    const int* __restrict__ skip_flag, i64 wstride) {
  Lout += (i64)blockIdx.y * wstride; A += (i64)blockIdx.y * wstride;
  Linv += (i64)blockIdx.y * wstride; Dinv += (i64)blockIdx.y * wstride;
  pdl_enter();
  if (skip_flag != nullptr && skip_flag[(i64)blockIdx.y * OS_SLOT_INTS] != 0) return;
  extern __shared__ __align__(16) float fin_smem[];
  const int nblk = (int)((sz + NB - 1) / NB);
  if ((int)blockIdx.x < nblk - 1) {   // the last row's last term (block column nblk - 2), and its finish
    inv_term(Lout, Linv, ld, Dinv, o, sz, nblk - 1, (int)blockIdx.x, nblk - 2, true, fin_smem);
    return;
  }
  const i64 total = sz * sz;
  const i64 first = (i64)((int)blockIdx.x - (nblk - 1)) * blockDim.x + threadIdx.x;
  const i64 step = (i64)((int)gridDim.x - (nblk - 1)) * blockDim.x;
  for (i64 e = first; e < total; e += step) {
    const i64 i = e / sz, c = e % sz;
    const i64 bi = i / NB, bc = c / NB;
    if (bi > bc) {
      A[(o + i) * ld + o + c] = Lout[(o + i) * ld + o + c];
    } else {
      Linv[(o + i) * ld + o + c] = (bi == bc) ? Dinv[((o + i) / NB) * (NB * NB) + (i % NB) * NB + (c % NB)] : 0.f;
    }
  }
}

// End of an adaptive round (one thread).  `minrel`, the smallest pivot relative to its
// column's squared norm, estimates 1 / cond^2 of the round's input panel.
//   - no pivot raised and minrel >= done_rel: the input was already orthonormal to
//     ~(1 - done_rel), so this round's output is orthonormal to rounding level: done;
//   - no pivot raised and minrel >= good_rel: cond <~ 1 / sqrt(good_rel); one more
//     round brings orthonormality to rounding level (the CholeskyQR2 argument), after
//     which the remaining rounds are skipped.
__global__ void k_round_end(int* __restrict__ os, float good_rel, float done_rel, int* __restrict__ rounds_total) {
  pdl_enter();
  os += (i64)blockIdx.x * OS_SLOT_INTS;
  if (os[OS_DONE] != 0) return;
  os[OS_ROUNDS] += 1;
  atomicAdd(rounds_total, 1);
  if (os[OS_GOOD] != 0) { os[OS_DONE] = 1; return; }
  const float minrel = __int_as_float(os[OS_MINREL]);
  if (os[OS_FLOORED] == 0) {
    if (minrel >= done_rel) os[OS_DONE] = 1;
    else if (minrel >= good_rel) os[OS_GOOD] = 1;
  }
}

// ---------------------------------------------------------------------------
// CholeskyQR2: is the first round's result U1 orthonormal enough to skip the second?  Measured without forming
// U1^T U1 (one third of the orthonormalization's tensor work): with NPROBE fixed sign vectors z_p (entries +-1
// from a hash of the index), E = U1^T U1 - I and w_p = U1^T (U1 z_p),  sum_p |w_p - z_p|^2 / NPROBE  is an
// unbiased estimate of |E|_F^2 (Hutchinson's estimator; relative spread sqrt(2 / NPROBE) per probe set at
// worst, far less for a matrix whose weight is spread over many entries).  Two passes over the panel.
// ---------------------------------------------------------------------------
constexpr int NPROBE = 8;

__device__ __forceinline__ float probe_sign(i64 j, int p) {
  uint32_t h = (uint32_t)j * 2654435761u + (uint32_t)(p + 1) * 0x9E3779B9u;
  h ^= h >> 15; h *= 2246822519u; h ^= h >> 13; h *= 3266489917u; h ^= h >> 16;
  return (h & 1u) ? 1.f : -1.f;
}

// Y[i][p] = sum_j U[i][j] z_p[j]: one warp per row (lanes stride over the columns).  grid = (blocks, matrices).
__global__ void __launch_bounds__(256) k_probe_y(const float* __restrict__ U, i64 ld, i64 rows, i64 r,
                                                 float* __restrict__ Y, i64 wstride, const int* __restrict__ keep) {
  pdl_enter();
  if (keep != nullptr && keep[(i64)blockIdx.y * OS_SLOT_INTS] != 0) return;   // this panel's decision stands
  U += (i64)blockIdx.y * wstride; Y += (i64)blockIdx.y * wstride;
  const int lane = threadIdx.x & 31;
  const i64 warp = (i64)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const i64 nwarps = (i64)gridDim.x * (blockDim.x >> 5);
  for (i64 i = warp; i < rows; i += nwarps) {
    float acc[NPROBE];
#pragma unroll
    for (int p = 0; p < NPROBE; ++p) acc[p] = 0.f;
    const float* urow = U + i * ld;
    for (i64 j = lane; j < r; j += 32) {
      const float u = urow[j];
#pragma unroll
      for (int p = 0; p < NPROBE; ++p) acc[p] = fmaf(u, probe_sign(j, p), acc[p]);
    }
#pragma unroll
    for (int p = 0; p < NPROBE; ++p) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc[p] += __shfl_xor_sync(0xffffffffu, acc[p], o);
    }
    if (lane == 0) {
#pragma unroll
      for (int p = 0; p < NPROBE; ++p) Y[i * NPROBE + p] = acc[p];
    }
  }
}

// The same for r a multiple of 4 (16-byte aligned rows): the +-1 entries of the probe vectors are hashed once per
// CTA and column block into a shared-memory table of floats instead of once per matrix element (the hash made the
// plain kernel ALU bound at a seventh of HBM speed), and a warp takes four rows at a time so that one read of a
// column's eight signs serves four elements.  Lane l owns columns 128 t + 4 l .. + 3 of a block of PY_COLS
// columns; wider panels add their later column blocks into Y (the same warp owns a row throughout).
constexpr int PY_COLS = 2048;
constexpr int PY_SMEM = PY_COLS * NPROBE * 4;
__global__ void __launch_bounds__(256) k_probe_y4(const float* __restrict__ U, i64 ld, i64 rows, i64 r,
                                                  float* __restrict__ Y, i64 wstride, const int* __restrict__ keep) {
  extern __shared__ __align__(16) float py_sign[];      // the signs of the block's columns (layout below)
  pdl_enter();
  if (keep != nullptr && keep[(i64)blockIdx.y * OS_SLOT_INTS] != 0) return;   // this panel's decision stands
  U += (i64)blockIdx.y * wstride; Y += (i64)blockIdx.y * wstride;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const i64 group0 = (i64)blockIdx.x * 8 + warp, groups = (i64)gridDim.x * 8;
  for (i64 c0 = 0; c0 < r; c0 += PY_COLS) {
    const int nc = (int)min((i64)PY_COLS, r - c0);
    __syncthreads();
    // table layout: the four signs (probes 4 h .. 4 h + 3) of column 128 t + 4 l + cc sit in the 16-byte unit
    // ((4 t + cc) 2 + h) 32 + l, so that the 32 lanes of a warp read 32 consecutive units (column-major by 8 floats
    // put a quarter warp's reads on the same banks: eight-way conflicts on every read)
    for (int e = threadIdx.x; e < nc * NPROBE; e += 256) {
      const int col = e / NPROBE, pr = e % NPROBE;
      py_sign[((((col >> 7) * 4 + (col & 3)) * 2 + (pr >> 2)) * 32 + ((col & 127) >> 2)) * 4 + (pr & 3)] = probe_sign(c0 + col, pr);
    }
    __syncthreads();
    for (i64 g = group0; g * 4 < rows; g += groups) {
      const i64 i0 = g * 4;
      float acc[4][NPROBE];
#pragma unroll
      for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int p = 0; p < NPROBE; ++p) acc[q][p] = 0.f;
      for (int j = 4 * lane; j < nc; j += 128) {
        float4 u[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          u[q] = (i0 + q < rows) ? *reinterpret_cast<const float4*>(U + (i0 + q) * ld + c0 + j) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          const float4* su = reinterpret_cast<const float4*>(py_sign) + (((j >> 7) * 4 + cc) * 2) * 32 + lane;
          const float4 s0 = su[0];
          const float4 s1 = su[32];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float v = (cc == 0) ? u[q].x : (cc == 1) ? u[q].y : (cc == 2) ? u[q].z : u[q].w;
            acc[q][0] = fmaf(v, s0.x, acc[q][0]); acc[q][1] = fmaf(v, s0.y, acc[q][1]);
            acc[q][2] = fmaf(v, s0.z, acc[q][2]); acc[q][3] = fmaf(v, s0.w, acc[q][3]);
            acc[q][4] = fmaf(v, s1.x, acc[q][4]); acc[q][5] = fmaf(v, s1.y, acc[q][5]);
            acc[q][6] = fmaf(v, s1.z, acc[q][6]); acc[q][7] = fmaf(v, s1.w, acc[q][7]);
          }
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int p = 0; p < NPROBE; ++p) {
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) acc[q][p] += __shfl_xor_sync(0xffffffffu, acc[q][p], o);
        }
      if (lane < 4 && i0 + lane < rows) {
        float* y = Y + (i0 + lane) * NPROBE;
#pragma unroll
        for (int p = 0; p < NPROBE; ++p) {
          const float v = (lane == 0) ? acc[0][p] : (lane == 1) ? acc[1][p] : (lane == 2) ? acc[2][p] : acc[3][p];
          y[p] = (c0 == 0) ? v : y[p] + v;
        }
      }
    }
  }
}

// part[chunk][j][p] = sum over the chunk's rows of U[i][j] Y[i][p].  grid = (ceil(r/128), chunks, matrices).
__global__ void __launch_bounds__(128) k_probe_w(const float* __restrict__ U, i64 ld, i64 rows, i64 r,
                                                 i64 rows_per_chunk, const float* __restrict__ Y,
                                                 float* __restrict__ part, i64 wstride, const int* __restrict__ keep) {
  pdl_enter();
  if (keep != nullptr && keep[(i64)blockIdx.z * OS_SLOT_INTS] != 0) return;
  U += (i64)blockIdx.z * wstride; Y += (i64)blockIdx.z * wstride; part += (i64)blockIdx.z * wstride;
  const i64 j = (i64)blockIdx.x * 128 + threadIdx.x;
  if (j >= r) return;
  const i64 i0 = (i64)blockIdx.y * rows_per_chunk;
  const i64 i1 = min(rows, i0 + rows_per_chunk);
  float acc[NPROBE];
#pragma unroll
  for (int p = 0; p < NPROBE; ++p) acc[p] = 0.f;
#pragma unroll 8      // (eight rows' loads in flight per thread; the sums keep their order)
  for (i64 i = i0; i < i1; ++i) {
    const float u = U[i * ld + j];
    const float4 y0 = *reinterpret_cast<const float4*>(Y + i * NPROBE);
    const float4 y1 = *reinterpret_cast<const float4*>(Y + i * NPROBE + 4);
    acc[0] = fmaf(u, y0.x, acc[0]); acc[1] = fmaf(u, y0.y, acc[1]); acc[2] = fmaf(u, y0.z, acc[2]); acc[3] = fmaf(u, y0.w, acc[3]);
    acc[4] = fmaf(u, y1.x, acc[4]); acc[5] = fmaf(u, y1.y, acc[5]); acc[6] = fmaf(u, y1.z, acc[6]); acc[7] = fmaf(u, y1.w, acc[7]);
  }
  float* out = part + ((i64)blockIdx.y * r + j) * NPROBE;
#pragma unroll
  for (int p = 0; p < NPROBE; ++p) out[p] = acc[p];
}

// The same for r a multiple of 4: a thread takes four neighbouring columns (one 16-byte load per row, four rows'
// loads in flight); every column's sum runs over the chunk's rows in the same order as above.
// grid = (ceil(r/512), chunks, matrices).
__global__ void __launch_bounds__(128) k_probe_w4(const float* __restrict__ U, i64 ld, i64 rows, i64 r,
                                                  i64 rows_per_chunk, const float* __restrict__ Y,
                                                  float* __restrict__ part, i64 wstride, const int* __restrict__ keep) {
  pdl_enter();
  if (keep != nullptr && keep[(i64)blockIdx.z * OS_SLOT_INTS] != 0) return;
  U += (i64)blockIdx.z * wstride; Y += (i64)blockIdx.z * wstride; part += (i64)blockIdx.z * wstride;
  const i64 j = ((i64)blockIdx.x * 128 + threadIdx.x) * 4;
  if (j >= r) return;
  const i64 i0 = (i64)blockIdx.y * rows_per_chunk;
  const i64 i1 = min(rows, i0 + rows_per_chunk);
  float acc[4][NPROBE];
#pragma unroll
  for (int c = 0; c < 4; ++c)
#pragma unroll
    for (int p = 0; p < NPROBE; ++p) acc[c][p] = 0.f;
#pragma unroll 4
  for (i64 i = i0; i < i1; ++i) {
    const float4 u4 = *reinterpret_cast<const float4*>(U + i * ld + j);
    const float4 y0 = *reinterpret_cast<const float4*>(Y + i * NPROBE);
    const float4 y1 = *reinterpret_cast<const float4*>(Y + i * NPROBE + 4);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float u = (c == 0) ? u4.x : (c == 1) ? u4.y : (c == 2) ? u4.z : u4.w;
      acc[c][0] = fmaf(u, y0.x, acc[c][0]); acc[c][1] = fmaf(u, y0.y, acc[c][1]);
      acc[c][2] = fmaf(u, y0.z, acc[c][2]); acc[c][3] = fmaf(u, y0.w, acc[c][3]);
      acc[c][4] = fmaf(u, y1.x, acc[c][4]); acc[c][5] = fmaf(u, y1.y, acc[c][5]);
      acc[c][6] = fmaf(u, y1.z, acc[c][6]); acc[c][7] = fmaf(u, y1.w, acc[c][7]);
    }
  }
  float4* out = reinterpret_cast<float4*>(part + ((i64)blockIdx.y * r + j) * NPROBE);
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    out[2 * c] = make_float4(acc[c][0], acc[c][1], acc[c][2], acc[c][3]);
    out[2 * c + 1] = make_float4(acc[c][4], acc[c][5], acc[c][6], acc[c][7]);
  }
}

// One block per matrix: est = sum_p |w_p - z_p|^2 / NPROBE (fixed summation order) into os[OS_MAXDEV] (float
// bits); est <= tau_f^2 * r  ->  the panel is done (OS_DONE = 1: the rest of the second round is skipped).
// Counts the rounds of the step that did work (1 or 2; with a recomputed panel 2 or 3).
// phase PROBE_FAST (the round ran on a panel from the fast product): done -> OS_DONE = 1, else 0 (a failed pivot
// too: the panel is recomputed before the fallback sees it); nothing is counted.  PROBE_AFTER_REDO: a panel that
// passed PROBE_FAST keeps its decision (one round); otherwise its recomputed first round is judged.
enum : int { PROBE_CHECK = 0, PROBE_FAST = 1, PROBE_AFTER_REDO = 2 };
__global__ void __launch_bounds__(1024) k_probe_decide(const float* __restrict__ part, int chunks, i64 r,
                                                      int* __restrict__ os, float tau_f,
                                                      int* __restrict__ rounds_total, i64 wstride, int phase) {
  pdl_enter();
  part += (i64)blockIdx.x * wstride;
  os += (i64)blockIdx.x * OS_SLOT_INTS;
  if (phase == PROBE_AFTER_REDO && os[OS_DONE] != 0) {
    if (threadIdx.x == 0) { os[OS_ROUNDS] = 1; atomicAdd(rounds_total, 1); }
    return;
  }
  __shared__ float red[1024];
  float e = 0.f;
  // one (column, probe) entry per thread at a time: consecutive threads read consecutive words of a chunk's partials
#pragma unroll 4       // (four entries' chunk sums advance together: their loads are independent)
  for (i64 x = threadIdx.x; x < r * NPROBE; x += blockDim.x) {
    float w = 0.f;
#pragma unroll 8      // (eight chunks' loads in flight; the sum keeps its order)
    for (int c = 0; c < chunks; ++c) w += part[(i64)c * r * NPROBE + x];
    const float dlt = w - probe_sign(x / NPROBE, (int)(x % NPROBE));
    e = fmaf(dlt, dlt, e);
  }
  red[threadIdx.x] = e;
  __syncthreads();
  for (int w = (int)blockDim.x / 2; w > 0; w >>= 1) {     // (the block size is a power of two)
    if ((int)threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float est = red[0] / (float)NPROBE;
    os[OS_MAXDEV] = __float_as_int(est);
    const bool failed = os[OS_FAIL] != 0;       // a pivot of the first round failed: the fallback redoes the panel
    const bool done = !failed && (est <= tau_f * tau_f * (float)r);      // false for NaN
    if (phase == PROBE_FAST) {
      os[OS_DONE] = done ? 1 : 0;
    } else {
      const int extra = (phase == PROBE_AFTER_REDO) ? 1 : 0;
      os[OS_DONE] = (done || failed) ? 1 : 0;
      os[OS_ROUNDS] = (done ? 1 : 2) + extra;
      atomicAdd(rounds_total, (done ? 1 : 2) + extra);
    }
  }
}

// Clears the round state of a step slot (keeps the fail flag): a second orthonormalization in one step.
__global__ void k_reset_rounds(int* __restrict__ os) {
  pdl_enter();
  os += (i64)blockIdx.x * OS_SLOT_INTS;
  os[OS_DONE] = 0; os[OS_GOOD] = 0; os[OS_FLOORED] = 0; os[OS_MAXDEV] = 0; os[OS_ROUNDS] = 0;
}

// After the last adaptive round: a panel that never became well conditioned is
// reported; if pivots were still being raised the step is cancelled (rank-deficient P).
__global__ void k_orth_finish(int* __restrict__ os, int* __restrict__ status) {
  pdl_enter();
  os += (i64)blockIdx.x * OS_SLOT_INTS;
  if (os[OS_DONE] != 0) return;
  if (os[OS_GOOD] == 0 && os[OS_FLOORED] != 0) {
    os[OS_FAIL] = 1;
    atomicOr(status, DION_STATUS_BREAKDOWN);
  } else {
    atomicOr(status, DION_STATUS_ILLCOND);
  }
}

// ---------------------------------------------------------------------------
// Fallback of Cholesky QR, on the device: when a pivot of CholeskyQR2 was not positive (the panel is too
// ill conditioned for the Gram matrix in fp32; the paper falls back to a QR factorization), the panel saved
// before the first round is orthonormalized column by column with classical Gram-Schmidt applied twice
// (the thin-QR factor with positive diagonal, like every other mode), in ONE cooperative launch that returns
// at once when no matrix of the chain failed: no host round trip, no launches beyond this one.
//
// CTA c owns a block of rows of the panel and only ever touches its own rows of U; what crosses CTAs are the
// partial dot products (part[c][k], summed in fixed CTA order into h[k]) and the partial squared norms,
// separated by grid-wide barriers (5 per column).  Column j, pass p: h_k = sum_i U[i][k] U[i][j] for k < j
// (pass 0 also k = j: the squared norm before orthogonalization), U[:, j] -= U[:, <j] h, then the norm and
// the scaling.  A column whose norm falls below CGS_DEFLATE_REL of what it was is linearly dependent on its
// predecessors to fp32 accuracy: the step is cancelled (OS_FAIL, DION_STATUS_BREAKDOWN) as before.
// Every barrier wait is bounded; when one runs out the kernel gives up with DION_STATUS_TIMEOUT and the step
// stays cancelled.
// ---------------------------------------------------------------------------
constexpr float CGS_DEFLATE_REL = 2e-6f;
constexpr int CGS_PASSES = 2;
constexpr int CGS_MAX_ROWS_PER_CTA = 1024;   // floats of shared memory for the CTA's piece of the current column

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Grid-wide barrier on a monotonic arrival counter: barrier number `epoch` (1, 2, ...) is passed when
// epoch * gridDim.x arrivals have been counted.  Returns false when the wait ran out or an earlier one did.
__device__ __forceinline__ bool cgs_grid_barrier(unsigned* counter, unsigned& epoch, long long limit, int* status,
                                                 volatile int* s_dead) {
  __syncthreads();
  ++epoch;
  if (threadIdx.x == 0 && !*s_dead) {
    __threadfence();
    atomicAdd(counter, 1u);
    const unsigned target = epoch * gridDim.x;
    const long long t0 = clock64();
    while (ld_acquire_u32(counter) < target) {
      if (clock64() - t0 > limit) {
        *s_dead = 1;
        atomicOr(status, DION_STATUS_TIMEOUT);
        break;
      }
      __nanosleep(100);
    }
    __threadfence();
  }
  __syncthreads();
  return *s_dead == 0;
}

__device__ __forceinline__ float cgs_block_sum(float v, float* red) {
  const int tid = threadIdx.x;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((tid & 31) == 0) red[tid >> 5] = v;
  __syncthreads();
  float t = 0.f;
  if (tid < 8) t = red[tid];
  if (tid < 32) {
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (tid == 0) red[8] = t;
  }
  __syncthreads();
  const float out = red[8];
  __syncthreads();
  return out;
}

// Pin: the saved panel (rows x r, ld); U: where the orthonormal factor goes (ld).  part: gridDim.x * r floats,
// hvec: r floats, npart: gridDim.x floats -- per matrix, wstride floats apart like every scratch offset.
__global__ void __launch_bounds__(256) k_cgs_fallback(const float* __restrict__ Pin, float* __restrict__ U, i64 ld,
                                                      i64 rows, i64 r, float* __restrict__ part, float* __restrict__ hvec,
                                                      float* __restrict__ npart, int* __restrict__ os_base,
                                                      int* __restrict__ status, int* __restrict__ fallbacks,
                                                      i64 wstride, int nb, long long spin_limit) {
  __shared__ float colj[CGS_MAX_ROWS_PER_CTA];
  __shared__ float red[9];
  __shared__ int s_dead;
  __shared__ float s_val;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = (int)gridDim.x, c = (int)blockIdx.x;
  const i64 rpc = (rows + G - 1) / G;
  const i64 i0 = min(rows, (i64)c * rpc), i1 = min(rows, i0 + rpc);
  const int nmy = (int)(i1 - i0);
  for (int b = 0; b < nb; ++b) {
    int* os = os_base + (i64)b * OS_SLOT_INTS;
    if (os[OS_FAIL] == 0) continue;                 // written by an earlier launch: every CTA reads the same value
    const float* Pb = Pin + (i64)b * wstride;
    float* Ub = U + (i64)b * wstride;
    float* partb = part + (i64)b * wstride;
    float* hb = hvec + (i64)b * wstride;
    float* nb_part = npart + (i64)b * wstride;
    unsigned* counter = reinterpret_cast<unsigned*>(os + OS_BARRIER);
    unsigned epoch = 0;
    if (tid == 0) s_dead = 0;
    __syncthreads();
    bool ok = true, deficient = false;
    for (i64 e = tid; e < (i64)nmy * r; e += 256) {
      const i64 i = i0 + e / r, k = e % r;
      Ub[i * ld + k] = Pb[i * ld + k];
    }
    __syncthreads();
    for (i64 j = 0; j < r && ok && !deficient; ++j) {
      for (int i = tid; i < nmy; i += 256) colj[i] = Ub[(i0 + i) * ld + j];
      __syncthreads();
      float before = 0.f;
      for (int pass = 0; pass < CGS_PASSES && ok; ++pass) {
        const i64 nk = j + (pass == 0 ? 1 : 0);     // pass 0: k = j is the squared norm before orthogonalization
        for (i64 k = tid; k < nk; k += 256) {
          float a0 = 0.f, a1 = 0.f;
          int i = 0;
          for (; i + 1 < nmy; i += 2) {
            a0 = fmaf(Ub[(i0 + i) * ld + k], colj[i], a0);
            a1 = fmaf(Ub[(i0 + i + 1) * ld + k], colj[i + 1], a1);
          }
          if (i < nmy) a0 = fmaf(Ub[(i0 + i) * ld + k], colj[i], a0);
          partb[(i64)c * r + k] = a0 + a1;
        }
        ok = cgs_grid_barrier(counter, epoch, spin_limit, status, &s_dead);
        if (!ok) break;
        {   // fixed-order sums over the CTAs, the k range split over the grid
          const i64 per = (nk + G - 1) / G;
          const i64 k0 = (i64)c * per, k1 = min(nk, k0 + per);
          for (i64 k = k0 + tid; k < k1; k += 256) {
            float sum = 0.f;
            for (int cc = 0; cc < G; ++cc) sum += partb[(i64)cc * r + k];
            hb[k] = sum;
          }
        }
        ok = cgs_grid_barrier(counter, epoch, spin_limit, status, &s_dead);
        if (!ok) break;
        if (pass == 0) before = hb[j];
        if (j > 0) {
          for (int i = warp; i < nmy; i += 8) {       // a warp per row: lanes stride over k
            const float* urow = Ub + (i0 + i) * ld;
            float acc = 0.f;
            for (i64 k = lane; k < j; k += 32) acc = fmaf(urow[k], hb[k], acc);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (lane == 0) colj[i] -= acc;
          }
          __syncthreads();
        }
      }
      if (!ok) break;
      float sq = 0.f;
      for (int i = tid; i < nmy; i += 256) sq = fmaf(colj[i], colj[i], sq);
      sq = cgs_block_sum(sq, red);
      if (tid == 0) nb_part[c] = sq;
      ok = cgs_grid_barrier(counter, epoch, spin_limit, status, &s_dead);
      if (!ok) break;
      if (tid == 0) {
        float tot = 0.f;
        for (int cc = 0; cc < G; ++cc) tot += nb_part[cc];
        s_val = tot;
      }
      __syncthreads();
      const float after = s_val;
      // every CTA sees the same two sums: the same decision everywhere
      if (!(after > CGS_DEFLATE_REL * CGS_DEFLATE_REL * before) || !(before < __int_as_float(0x7f800000))) {
        deficient = true;
        break;
      }
      const float inv = rsqrtf(after);
      for (int i = tid; i < nmy; i += 256) Ub[(i0 + i) * ld + j] = colj[i] * inv;
      __syncthreads();
    }
    if (c == 0 && tid == 0) {
      if (ok && !deficient) {
        os[OS_FAIL] = 0;
        atomicAdd(fallbacks, 1);
      } else {
        os[OS_FAIL] = 1;
        if (deficient) atomicOr(status, DION_STATUS_BREAKDOWN);
      }
    }
    __syncthreads();
  }
}

// Copies a rows x cols block between two matrices (leading dimensions lds, ldd).
__global__ void k_copy_block(const float* __restrict__ src, i64 lds, float* __restrict__ dst, i64 ldd,
                             i64 rows, i64 cols, const int* __restrict__ skip_flag, i64 wstride) {
  pdl_enter();
  src += (i64)blockIdx.y * wstride; dst += (i64)blockIdx.y * wstride;     // batched over blockIdx.y
  if (skip_flag != nullptr && skip_flag[(i64)blockIdx.y * OS_SLOT_INTS] != 0) return;
  const i64 total = rows * cols;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / cols, c = e % cols;
    dst[i * ldd + c] = src[i * lds + c];
  }
}

// Partial sums of squares per column: part[chunk][j] = sum over the chunk's rows of R[i][j]^2.
// grid = (ceil(r/128), chunks); 128 threads, one column each (coalesced rows).
__global__ void __launch_bounds__(128) k_colsumsq_partial(const float* __restrict__ R, i64 ld, i64 n, i64 r,
                                                          i64 rows_per_chunk, float* __restrict__ part,
                                                          const int* __restrict__ skip_flag, i64 wstride) {
  // blockIdx.z: the matrix of a chain (R and part wstride floats apart, skip flags a state slot apart)
  pdl_enter();
  if (skip_flag != nullptr && skip_flag[(i64)blockIdx.z * OS_SLOT_INTS] != 0) return;
  R += (i64)blockIdx.z * wstride; part += (i64)blockIdx.z * wstride;
  const i64 j = (i64)blockIdx.x * 128 + threadIdx.x;
  if (j >= r) return;
  const i64 i0 = (i64)blockIdx.y * rows_per_chunk;
  const i64 i1 = min(n, i0 + rows_per_chunk);
  float s = 0.f;
  for (i64 i = i0; i < i1; ++i) {
    const float v = R[i * ld + j];
    s = fmaf(v, v, s);
  }
  part[(i64)blockIdx.y * r + j] = s;
}

// out[j] = sum over the chunks (in order) of part[chunk][j]: the squared column norms of a shard's rows,
// handed to the caller for the all-reduce over the shards (1D-sharded Dion).
__global__ void __launch_bounds__(128) k_colsumsq_finish(const float* __restrict__ part, int chunks, i64 r,
                                                         float* __restrict__ out, const int* __restrict__ skip_flag) {
  pdl_enter();
  if (skip_flag != nullptr && *skip_flag != 0) return;
  const i64 j = (i64)blockIdx.x * 128 + threadIdx.x;
  if (j >= r) return;
  float s = 0.f;
  for (int c = 0; c < chunks; ++c) s += part[(i64)c * r + j];
  out[j] = s;
}

// ColNorm: d_j = sqrt(sum of the partials in chunk order); Q[i][j] = R[i][j] / (d_j + eps).
// Same grid as k_colsumsq_partial.  The chunk-0 blocks also export d.
__global__ void __launch_bounds__(128) k_colnorm_apply(const float* __restrict__ R, i64 ldr, i64 n, i64 r,
                                                       i64 rows_per_chunk, int chunks,
                                                       const float* __restrict__ part, float eps,
                                                       float* __restrict__ Q, i64 ldq,
                                                       float* __restrict__ d_ws, float* __restrict__ d_out,
                                                       int* __restrict__ status,
                                                       const int* __restrict__ skip_flag, i64 wstride,
                                                       const ChainPtrs Qs, const ChainPtrs ds) {
  // wstride != 0: one launch over a chain (blockIdx.z): R, part and d_ws in the scratch slices, Q and d_out from
  // the pointer tables
  pdl_enter();
  if (skip_flag != nullptr && skip_flag[(i64)blockIdx.z * OS_SLOT_INTS] != 0) return;
  if (wstride != 0) {
    R += (i64)blockIdx.z * wstride; part += (i64)blockIdx.z * wstride; d_ws += (i64)blockIdx.z * wstride;
    Q = reinterpret_cast<float*>(const_cast<void*>(Qs.p[blockIdx.z]));
    d_out = reinterpret_cast<float*>(const_cast<void*>(ds.p[blockIdx.z]));
  }
  const i64 j = (i64)blockIdx.x * 128 + threadIdx.x;
  if (j >= r) return;
  float s = 0.f;
  for (int c = 0; c < chunks; ++c) s += part[(i64)c * r + j];
  const float d = sqrtf(s);
  if (blockIdx.y == 0) {
    d_ws[j] = d;
    if (d_out != nullptr) d_out[j] = d;
    if (!isfinite(d)) atomicOr(status, DION_STATUS_NONFINITE);
  }
  const float inv = 1.f / (d + eps);
  const i64 i0 = (i64)blockIdx.y * rows_per_chunk;
  const i64 i1 = min(n, i0 + rows_per_chunk);
  for (i64 i = i0; i < i1; ++i) Q[i * ldq + j] = R[i * ldr + j] * inv;
}

// Copies a rows x r panel (ld = ldv) into Q (ld = ldq) unless the step was flagged.
// `only_if` (optional): the copy happens only when *only_if != 0.
__global__ void k_copy_panel(const float* __restrict__ V, i64 ldv, float* __restrict__ Q, i64 ldq,
                             i64 rows, i64 r, const int* __restrict__ skip_flag,
                             const int* __restrict__ only_if, i64 wstride) {
  pdl_enter();
  V += (i64)blockIdx.y * wstride;                                         // batched over blockIdx.y
  if (wstride != 0) Q += (i64)blockIdx.y * wstride;
  if (skip_flag != nullptr && skip_flag[(i64)blockIdx.y * OS_SLOT_INTS] != 0) return;
  if (only_if != nullptr && only_if[(i64)blockIdx.y * OS_SLOT_INTS] == 0) return;
  const i64 total = rows * r;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / r, c = e % r;
    Q[i * ldq + c] = V[i * ldv + c];
  }
}

// *dst = 1 if *src != 0 (carries a breakdown from one call of a multi-call step to the next).
__global__ void k_latch_flag(const int* __restrict__ src, int* __restrict__ dst) {
  pdl_enter();
  if (*src != 0) *dst = 1;
}

// Counts a skipped step (breakdown) at the end of a step's launch chain.
__global__ void k_finish_step(const int* __restrict__ step_flag, int* __restrict__ skipped) {
  pdl_enter();
  if (step_flag[(i64)blockIdx.x * OS_SLOT_INTS] != 0) atomicAdd(skipped, 1);
}

// ---------------------------------------------------------------------------
// Householder QR (unblocked), the slow robust mode.
// ---------------------------------------------------------------------------

// Column j: builds the unit reflector v (stored in V[j:, j]) from A[j:, j] and
// records R_qr[j][j] = alpha in diag[j].  One block of 1024 threads.
__global__ void __launch_bounds__(1024) k_hh_reflector(float* __restrict__ A, i64 lda, i64 m, i64 j,
                                                       float* __restrict__ V, i64 ldv,
                                                       float* __restrict__ diag) {
  __shared__ float red[1024];
  __shared__ float s_alpha, s_vnorm;
  const int tid = threadIdx.x;
  float s = 0.f;
  for (i64 i = j + tid; i < m; i += 1024) { const float v = A[i * lda + j]; s = fmaf(v, v, s); }
  red[tid] = s;
  __syncthreads();
  for (int w = 512; w > 0; w >>= 1) { if (tid < w) red[tid] += red[tid + w]; __syncthreads(); }
  if (tid == 0) {
    const float norm = sqrtf(red[0]);
    const float a0 = A[j * lda + j];
    const float alpha = (a0 >= 0.f) ? -norm : norm;
    // ||x - alpha e1||^2 = 2 norm^2 + 2 norm |x0|
    s_alpha = alpha;
    s_vnorm = sqrtf(2.f * norm * (norm + fabsf(a0)));
    diag[j] = alpha;
  }
  __syncthreads();
  const float alpha = s_alpha, vn = s_vnorm;
  for (i64 i = j + tid; i < m; i += 1024) {
    float v = A[i * lda + j];
    if (i == j) v -= alpha;
    V[i * ldv + j] = (vn > 0.f) ? v / vn : 0.f;
  }
}

// T[j0:, c] -= 2 v (v^T T[j0:, c]) for the columns c in [c_begin, c_end); v = V[j0:, vj].
// grid.x = column chunks of 32; block = 32 x 8 (32 columns, 8 row lanes).
__global__ void __launch_bounds__(256) k_hh_apply(float* __restrict__ T, i64 ldt, i64 m, i64 j0,
                                                  const float* __restrict__ V, i64 ldv, i64 vj,
                                                  i64 c_begin, i64 c_end) {
  __shared__ float red[8][33];
  const int cx = threadIdx.x % 32, ry = threadIdx.x / 32;
  const i64 c = c_begin + (i64)blockIdx.x * 32 + cx;
  const bool ok = c < c_end;
  float s = 0.f;
  if (ok) for (i64 i = j0 + ry; i < m; i += 8) s = fmaf(V[i * ldv + vj], T[i * ldt + c], s);
  red[ry][cx] = s;
  __syncthreads();
  float w = 0.f;
#pragma unroll
  for (int k = 0; k < 8; ++k) w += red[k][cx];
  w *= 2.f;
  if (ok) for (i64 i = j0 + ry; i < m; i += 8) T[i * ldt + c] = fmaf(-V[i * ldv + vj], w, T[i * ldt + c]);
}

// U = first r columns of the identity.
__global__ void k_set_identity(float* __restrict__ U, i64 ld, i64 m, i64 r) {
  const i64 total = m * r;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / r, c = e % r;
    U[i * ld + c] = (i == c) ? 1.f : 0.f;
  }
}

// Sign convention: negate column j of U wherever diag[j] (= R_qr[j][j]) < 0.
__global__ void k_sign_fix(float* __restrict__ U, i64 ld, i64 m, i64 r, const float* __restrict__ diag) {
  const i64 total = m * r;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / r, c = e % r;
    if (diag[c] < 0.f) U[i * ld + c] = -U[i * ld + c];
  }
}

}  // namespace dion

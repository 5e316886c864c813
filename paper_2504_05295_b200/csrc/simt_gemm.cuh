// fp32 FMA tiled product with fused operand formation and epilogues.
// Takes any shape, stride and alignment; it is the engine for small or ragged
// problems and for the r x r factor updates, and the reference engine the
// tensor-core kernels are compared with.
#pragma once

#include "dion_common.cuh"

namespace dion {

template <int BM, int BN, int BK, int TM, int TN>
__global__ void __launch_bounds__(256) k_gemm_simt(const GemmArgs g) {
  pdl_enter();
  static_assert((BM / TM) * (BN / TN) == 256, "256 threads per tile");
  static_assert(TM % 4 == 0 && TN % 4 == 0, "micro tile in groups of 4");
  // blockIdx.z = inner batch index + batch * outer batch index (or the K split)
  i64 batch = 0, outer = 0;
  int split = 0;
  if (g.splits > 1) split = blockIdx.z;
  else { batch = blockIdx.z % g.batch; outer = blockIdx.z / g.batch; }
  if (g.skip_flag != nullptr && g.skip_flag[outer * g.skip_stride] != 0) return;

  constexpr int LDA_S = BM + 4, LDB_S = BN + 4;
  constexpr int A_PER = BM * BK / 256, B_PER = BN * BK / 256;
  constexpr int GM = TM / 4, GN = TN / 4;          // groups of 4 rows / cols per thread
  constexpr int SM_STRIDE = BM / GM, SN_STRIDE = BN / GN;
  __shared__ __align__(16) float As[BK][LDA_S];
  __shared__ __align__(16) float Bs[BK][LDB_S];

  const int tid = threadIdx.x;
  const int tx = tid % (BN / TN), ty = tid / (BN / TN);
  const i64 i0 = (i64)blockIdx.y * BM, j0 = (i64)blockIdx.x * BN;
  if (g.tri == TRI_LOWER && j0 > i0 + BM - 1) return;

  i64 k_begin = 0, k_end = g.K;
  if (g.klimit) k_end = min(g.K, j0 + BN);
  if (g.splits > 1) {
    i64 per = (g.K + g.splits - 1) / g.splits;
    per = (per + BK - 1) / BK * BK;
    k_begin = min(g.K, per * split);
    k_end = min(k_end, k_begin + per);
  }

  const float* A = g.A + batch * g.bsA + outer * g.bs2;
  const float* B = g.B + batch * g.bsB + outer * g.bs2;
  const bool a_kcontig = (g.a_sk == 1);
  const bool b_ncontig = (g.b_sn == 1);

  float acc[TM][TN];
#pragma unroll
  for (int a = 0; a < TM; ++a)
#pragma unroll
    for (int b = 0; b < TN; ++b) acc[a][b] = 0.f;

  float ra[A_PER], rb[B_PER];

  auto fetch = [&](i64 kb) {
#pragma unroll
    for (int l = 0; l < A_PER; ++l) {
      const int idx = tid + l * 256;
      const int ii = a_kcontig ? idx / BK : idx % BM;
      const int kk = a_kcontig ? idx % BK : idx / BM;
      const i64 gi = i0 + ii, gk = kb + kk;
      float v = 0.f;
      if (gi < g.M && gk < k_end) {
        v = A[gi * g.a_si + gk * g.a_sk];
        if (g.a2_mode != ADD_NONE) v += load_add(g.A2, gi * g.a2_si + gk * g.a2_sk, g.a2_mode);
      }
      ra[l] = v;
    }
#pragma unroll
    for (int l = 0; l < B_PER; ++l) {
      const int idx = tid + l * 256;
      const int jj = b_ncontig ? idx % BN : idx / BK;
      const int kk = b_ncontig ? idx / BN : idx % BK;
      const i64 gj = j0 + jj, gk = kb + kk;
      float v = 0.f;
      if (gj < g.N && gk < k_end) v = B[gk * g.b_sk + gj * g.b_sn];
      rb[l] = v;
    }
  };
  auto stage = [&]() {
#pragma unroll
    for (int l = 0; l < A_PER; ++l) {
      const int idx = tid + l * 256;
      const int ii = a_kcontig ? idx / BK : idx % BM;
      const int kk = a_kcontig ? idx % BK : idx / BM;
      As[kk][ii] = ra[l];
    }
#pragma unroll
    for (int l = 0; l < B_PER; ++l) {
      const int idx = tid + l * 256;
      const int jj = b_ncontig ? idx % BN : idx / BK;
      const int kk = b_ncontig ? idx / BN : idx % BK;
      Bs[kk][jj] = rb[l];
    }
  };

  if (k_begin < k_end) fetch(k_begin);
  for (i64 kb = k_begin; kb < k_end; kb += BK) {
    stage();
    __syncthreads();
    if (kb + BK < k_end) fetch(kb + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[TM], b[TN];
#pragma unroll
      for (int gm = 0; gm < GM; ++gm) {
        const float4 v = *reinterpret_cast<const float4*>(&As[kk][gm * SM_STRIDE + ty * 4]);
        a[gm * 4 + 0] = v.x; a[gm * 4 + 1] = v.y; a[gm * 4 + 2] = v.z; a[gm * 4 + 3] = v.w;
      }
#pragma unroll
      for (int gn = 0; gn < GN; ++gn) {
        const float4 v = *reinterpret_cast<const float4*>(&Bs[kk][gn * SN_STRIDE + tx * 4]);
        b[gn * 4 + 0] = v.x; b[gn * 4 + 1] = v.y; b[gn * 4 + 2] = v.z; b[gn * 4 + 3] = v.w;
      }
#pragma unroll
      for (int x = 0; x < TM; ++x)
#pragma unroll
        for (int y = 0; y < TN; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
    }
    __syncthreads();
  }

  float alpha = g.alpha;
  if (g.alpha_dev != nullptr) alpha *= *g.alpha_dev;

  if (g.splits > 1) {
    float* part = g.part + (i64)split * g.M * g.N;
#pragma unroll
    for (int x = 0; x < TM; ++x) {
      const i64 gi = i0 + (x / 4) * SM_STRIDE + ty * 4 + (x % 4);
      if (gi >= g.M) continue;
#pragma unroll
      for (int y = 0; y < TN; ++y) {
        const i64 gj = j0 + (y / 4) * SN_STRIDE + tx * 4 + (y % 4);
        if (gj < g.N) part[gi * g.N + gj] = acc[x][y];
      }
    }
    return;
  }

  float* C = g.C + batch * g.bsC + outer * g.bs2;
#pragma unroll
  for (int x = 0; x < TM; ++x) {
    const i64 gi = i0 + (x / 4) * SM_STRIDE + ty * 4 + (x % 4);
    if (gi >= g.M) continue;
#pragma unroll
    for (int y = 0; y < TN; ++y) {
      const i64 gj = j0 + (y / 4) * SN_STRIDE + tx * 4 + (y % 4);
      if (gj >= g.N) continue;
      float* c = C + gi * g.ldc + gj;
      const float v = alpha * acc[x][y];
      if (g.epi == EPI_STORE) {
        *c = v;
      } else if (g.epi == EPI_SUB) {
        *c = *c - v;
      } else if (g.epi == EPI_C2_SUB) {
        *c = load_add(g.C2, gi * g.ldc2 + gj, ADD_F32) - v;
      } else {
        *c = (*c + load_add(g.C2, gi * g.ldc2 + gj, g.c2_mode)) - v;
      }
    }
  }
}

// Sums split-K partials in a fixed order: C = alpha * sum_s part[s].
__global__ void k_splitk_reduce(const float* __restrict__ part, int splits, i64 M, i64 N,
                                float* __restrict__ C, i64 ldc, float alpha, int tri, int tile,
                                const int* skip_flag, i64 bstride, i64 skip_stride,
                                const float* __restrict__ alpha_dev = nullptr, i64 alpha_dev_stride = 0) {
  // blockIdx.y: the matrix of a batched product (partials and output bstride elements apart)
  pdl_enter();
  if (skip_flag != nullptr && skip_flag[(i64)blockIdx.y * skip_stride] != 0) return;
  if (alpha_dev != nullptr) alpha *= alpha_dev[(i64)blockIdx.y * alpha_dev_stride];
  part += (i64)blockIdx.y * bstride;
  C += (i64)blockIdx.y * bstride;
  const i64 total = M * N;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / N, j = e % N;
    if (tri == TRI_LOWER && (j / tile) > (i / tile)) continue;  // tiles that were never computed
    float s = 0.f;
    for (int p = 0; p < splits; ++p) s += part[(i64)p * total + e];
    C[i * ldc + j] = alpha * s;
  }
}

}  // namespace dion

// Operand preparation in scratch: bf16(M + G) and bf16 copies (bf16-operand mode), M + G in fp32, and
// TF32-rounded copies of the factors of the weight update (fp32 mode).
#pragma once

#include <cuda_fp16.h>

#include "dion_common.cuh"

namespace dion {

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// B16 = bf16(M + G), rows x cols, B16 dense with leading dimension cols (a multiple of 8).
// One thread per 8 consecutive elements of a row.  VEC: M (and G) rows start 16-byte
// aligned (pointer and leading dimension), so the loads are 128-bit.
template <bool VEC>
__global__ void __launch_bounds__(256) k_form_b16(const float* __restrict__ M, i64 ldm, const void* __restrict__ G,
                                                  i64 ldg, int g_mode, i64 rows, i64 cols,
                                                  __nv_bfloat16* __restrict__ out) {
  pdl_enter();
  const i64 per_row = cols / 8;
  const i64 total = rows * per_row;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / per_row, c = (e - i * per_row) * 8;
    float v[8];
    const float* mp = M + i * ldm + c;
    if (VEC) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(mp)), b = __ldg(reinterpret_cast<const float4*>(mp) + 1);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = mp[q];
    }
    if (g_mode == ADD_F32) {
      const float* gp = reinterpret_cast<const float*>(G) + i * ldg + c;
      if (VEC) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(gp)), b = __ldg(reinterpret_cast<const float4*>(gp) + 1);
        v[0] += a.x; v[1] += a.y; v[2] += a.z; v[3] += a.w; v[4] += b.x; v[5] += b.y; v[6] += b.z; v[7] += b.w;
      } else {
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] += gp[q];
      }
    } else if (g_mode == ADD_BF16) {
      const __nv_bfloat16* gp = reinterpret_cast<const __nv_bfloat16*>(G) + i * ldg + c;
      if (VEC) {
        const uint4 w = __ldg(reinterpret_cast<const uint4*>(gp));
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const __nv_bfloat162 h = *reinterpret_cast<const __nv_bfloat162*>(&ww[q]);
          v[2 * q] += __low2float(h); v[2 * q + 1] += __high2float(h);
        }
      } else {
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] += __bfloat162float(gp[q]);
      }
    }
    uint4 o;
    o.x = pack_bf16x2(v[0], v[1]); o.y = pack_bf16x2(v[2], v[3]);
    o.z = pack_bf16x2(v[4], v[5]); o.w = pack_bf16x2(v[6], v[7]);
    *reinterpret_cast<uint4*>(out + i * cols + c) = o;
  }
}

// B32 = M + G in fp32, rows x cols (cols a multiple of 4), B32 dense with leading dimension cols: the sum the
// fused operand formation of the contraction kernel computes, formed once per step where two products and the
// error feedback read it.  One thread per 4 consecutive elements of a row; VEC as above.
// hi / lo (optional, both or neither; cols a multiple of 8 then): the same sum as a pair of bf16 arrays, hi = bf16(sum),
// lo = bf16(sum - hi), dense like out: the operand of the products that run on bf16 pairs.
template <bool VEC>
__device__ __forceinline__ void form_b32_body(const float* __restrict__ M, i64 ldm, const void* __restrict__ G,
                                              i64 ldg, int g_mode, i64 rows, i64 cols, float* __restrict__ out,
                                              __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
  const i64 per_row = cols / 4;
  const i64 total = rows * per_row;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / per_row, c = (e - i * per_row) * 4;
    float4 v;
    const float* mp = M + i * ldm + c;
    if (VEC) v = __ldg(reinterpret_cast<const float4*>(mp));
    else v = make_float4(mp[0], mp[1], mp[2], mp[3]);
    if (g_mode == ADD_F32) {
      const float* gp = reinterpret_cast<const float*>(G) + i * ldg + c;
      float4 g;
      if (VEC) g = __ldg(reinterpret_cast<const float4*>(gp));
      else g = make_float4(gp[0], gp[1], gp[2], gp[3]);
      v.x += g.x; v.y += g.y; v.z += g.z; v.w += g.w;
    } else if (g_mode == ADD_BF16) {
      const __nv_bfloat16* gp = reinterpret_cast<const __nv_bfloat16*>(G) + i * ldg + c;
      if (VEC) {
        const uint2 w = __ldg(reinterpret_cast<const uint2*>(gp));
        const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&w.x);
        const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&w.y);
        v.x += __low2float(lo); v.y += __high2float(lo); v.z += __low2float(hi); v.w += __high2float(hi);
      } else {
        v.x += __bfloat162float(gp[0]); v.y += __bfloat162float(gp[1]);
        v.z += __bfloat162float(gp[2]); v.w += __bfloat162float(gp[3]);
      }
    }
    *reinterpret_cast<float4*>(out + i * cols + c) = v;
    if (hi != nullptr) {
      const float h0 = __bfloat162float(__float2bfloat16_rn(v.x)), h1 = __bfloat162float(__float2bfloat16_rn(v.y));
      const float h2 = __bfloat162float(__float2bfloat16_rn(v.z)), h3 = __bfloat162float(__float2bfloat16_rn(v.w));
      uint2 oh, ol;
      oh.x = pack_bf16x2(h0, h1); oh.y = pack_bf16x2(h2, h3);
      ol.x = pack_bf16x2(v.x - h0, v.y - h1); ol.y = pack_bf16x2(v.z - h2, v.w - h3);
      *reinterpret_cast<uint2*>(hi + i * cols + c) = oh;
      *reinterpret_cast<uint2*>(lo + i * cols + c) = ol;
    }
  }
}
template <bool VEC>
__global__ void __launch_bounds__(256) k_form_b32(const float* __restrict__ M, i64 ldm, const void* __restrict__ G,
                                                  i64 ldg, int g_mode, i64 rows, i64 cols, float* __restrict__ out,
                                                  __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
  pdl_enter();
  form_b32_body<VEC>(M, ldm, G, ldg, g_mode, rows, cols, out, hi, lo);
}
// The same for every matrix of a chain in one launch (blockIdx.y): the caller's M and G from pointer tables, the
// outputs in the scratch slices, `ostride` floats apart.
template <bool VEC>
__global__ void __launch_bounds__(256) k_form_b32_chain(const ChainPtrs Ms, i64 ldm, const ChainPtrs Gs, i64 ldg, int g_mode,
                                                        i64 rows, i64 cols, float* __restrict__ out,
                                                        __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                        i64 ostride) {
  pdl_enter();
  const i64 b = blockIdx.y;
  form_b32_body<VEC>(reinterpret_cast<const float*>(Ms.p[b]), ldm, Gs.p[b], ldg, g_mode, rows, cols, out + b * ostride,
                     hi != nullptr ? hi + 2 * b * ostride : nullptr, lo != nullptr ? lo + 2 * b * ostride : nullptr);
}

// out = bf16(src), rows x cols (cols a multiple of 8, src rows 16-byte aligned), out dense.
// skip_flag (optional): nothing is written when *skip_flag != 0.
__global__ void __launch_bounds__(256) k_to_bf16(const float* __restrict__ src, i64 lds, i64 rows, i64 cols,
                                                 __nv_bfloat16* __restrict__ out, const int* __restrict__ skip_flag) {
  pdl_enter();
  if (skip_flag != nullptr && *skip_flag != 0) return;
  const i64 per_row = cols / 8;
  const i64 total = rows * per_row;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / per_row, c = (e - i * per_row) * 8;
    const float4 a = *reinterpret_cast<const float4*>(src + i * lds + c);
    const float4 b = *(reinterpret_cast<const float4*>(src + i * lds + c) + 1);
    uint4 o;
    o.x = pack_bf16x2(a.x, a.y); o.y = pack_bf16x2(a.z, a.w);
    o.z = pack_bf16x2(b.x, b.y); o.w = pack_bf16x2(b.z, b.w);
    *reinterpret_cast<uint4*>(out + i * cols + c) = o;
  }
}

// hi = bf16(src), lo = bf16(src - hi): src ~ hi + lo to 16 significant bits.  rows x cols (cols a multiple of 8,
// src rows 16-byte aligned), hi and lo dense.  skip_flag (optional): nothing is written when *skip_flag != 0.
// copy (optional): src also as a dense fp32 array
__device__ __forceinline__ void split_bf16_body(const float* __restrict__ src, i64 lds, i64 rows, i64 cols,
                                                __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                float* __restrict__ copy = nullptr) {
  const i64 per_row = cols / 8;
  const i64 total = rows * per_row;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / per_row, c = (e - i * per_row) * 8;
    const float4 a = *reinterpret_cast<const float4*>(src + i * lds + c);
    const float4 b = *(reinterpret_cast<const float4*>(src + i * lds + c) + 1);
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    float h[8], l[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      h[q] = __bfloat162float(__float2bfloat16_rn(v[q]));
      l[q] = v[q] - h[q];
    }
    uint4 oh, ol;
    oh.x = pack_bf16x2(h[0], h[1]); oh.y = pack_bf16x2(h[2], h[3]); oh.z = pack_bf16x2(h[4], h[5]); oh.w = pack_bf16x2(h[6], h[7]);
    ol.x = pack_bf16x2(l[0], l[1]); ol.y = pack_bf16x2(l[2], l[3]); ol.z = pack_bf16x2(l[4], l[5]); ol.w = pack_bf16x2(l[6], l[7]);
    *reinterpret_cast<uint4*>(hi + i * cols + c) = oh;
    *reinterpret_cast<uint4*>(lo + i * cols + c) = ol;
    if (copy != nullptr) {
      *reinterpret_cast<float4*>(copy + i * cols + c) = a;
      *(reinterpret_cast<float4*>(copy + i * cols + c) + 1) = b;
    }
  }
}
__global__ void __launch_bounds__(256) k_split_bf16(const float* __restrict__ src, i64 lds, i64 rows, i64 cols,
                                                    __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                    const int* __restrict__ skip_flag) {
  pdl_enter();
  if (skip_flag != nullptr && *skip_flag != 0) return;
  split_bf16_body(src, lds, rows, cols, hi, lo);
}
// One launch over the matrices of a chain (blockIdx.y): sources from a pointer table, outputs `ostride` floats
// apart in the scratch slices, skip flags `skip_stride` ints apart.
__global__ void __launch_bounds__(256) k_split_bf16_chain(const ChainPtrs srcs, i64 lds, i64 rows, i64 cols,
                                                          __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                          i64 ostride, const int* __restrict__ skip_flag, i64 skip_stride,
                                                          float* __restrict__ copy) {
  pdl_enter();
  const i64 b = blockIdx.y;
  if (skip_flag != nullptr && skip_flag[b * skip_stride] != 0) return;
  split_bf16_body(reinterpret_cast<const float*>(srcs.p[b]), lds, rows, cols, hi + 2 * b * ostride, lo + 2 * b * ostride,
                  copy != nullptr ? copy + b * ostride : nullptr);
}

// out = src with every value rounded to the nearest TF32 number (10 explicit mantissa bits, ties away
// from zero), rows x cols (cols a multiple of 4, src rows 16-byte aligned), out dense.  The tensor core
// truncates an fp32 operand to TF32 when it reads it; on pre-rounded values that truncation is exact, so a
// single-pass TF32 product of such arrays carries an unbiased operand error of at most 2^-11 relative.
// skip_flag (optional): nothing is written when *skip_flag != 0.
__device__ __forceinline__ void round_tf32_body(const float* __restrict__ src, i64 lds, i64 rows, i64 cols,
                                                float* __restrict__ out) {
  const i64 per_row = cols / 4;
  const i64 total = rows * per_row;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / per_row, c = (e - i * per_row) * 4;
    const float4 a = *reinterpret_cast<const float4*>(src + i * lds + c);
    uint4 o;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(o.x) : "f"(a.x));
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(o.y) : "f"(a.y));
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(o.z) : "f"(a.z));
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(o.w) : "f"(a.w));
    *reinterpret_cast<uint4*>(out + i * cols + c) = o;
  }
}
__global__ void __launch_bounds__(256) k_round_tf32(const float* __restrict__ src, i64 lds, i64 rows, i64 cols,
                                                    float* __restrict__ out, const int* __restrict__ skip_flag) {
  pdl_enter();
  if (skip_flag != nullptr && *skip_flag != 0) return;
  round_tf32_body(src, lds, rows, cols, out);
}
__global__ void __launch_bounds__(256) k_round_tf32_chain(const ChainPtrs srcs, i64 lds, i64 rows, i64 cols,
                                                          float* __restrict__ out, i64 ostride,
                                                          const int* __restrict__ skip_flag, i64 skip_stride) {
  pdl_enter();
  const i64 b = blockIdx.y;
  if (skip_flag != nullptr && skip_flag[b * skip_stride] != 0) return;
  round_tf32_body(reinterpret_cast<const float*>(srcs.p[b]), lds, rows, cols, out + b * ostride);
}

// out = half(scale * src), round to nearest: the factors of the weight update as IEEE half arrays (11 significant
// bits, like TF32, at the 16-bit MMA rate and half the operand bytes).  `scale` is a power of two chosen by the caller
// so that entries of a matrix with unit-norm columns sit around 1: far from half's subnormals, and at most
// sqrt(2 rows) < 65504.  rows x cols (cols a multiple of 8, src rows 16-byte aligned), out dense.
__device__ __forceinline__ void round_f16_body(const float* __restrict__ src, i64 lds, i64 rows, i64 cols, float scale,
                                               __half* __restrict__ out) {
  const i64 per_row = cols / 8;
  const i64 total = rows * per_row;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / per_row, c = (e - i * per_row) * 8;
    const float4 a = *reinterpret_cast<const float4*>(src + i * lds + c);
    const float4 b = *(reinterpret_cast<const float4*>(src + i * lds + c) + 1);
    __half2 h0 = __floats2half2_rn(scale * a.x, scale * a.y), h1 = __floats2half2_rn(scale * a.z, scale * a.w);
    __half2 h2 = __floats2half2_rn(scale * b.x, scale * b.y), h3 = __floats2half2_rn(scale * b.z, scale * b.w);
    uint4 o;
    o.x = *reinterpret_cast<uint32_t*>(&h0); o.y = *reinterpret_cast<uint32_t*>(&h1);
    o.z = *reinterpret_cast<uint32_t*>(&h2); o.w = *reinterpret_cast<uint32_t*>(&h3);
    *reinterpret_cast<uint4*>(out + i * cols + c) = o;
  }
}
__global__ void __launch_bounds__(256) k_round_f16(const float* __restrict__ src, i64 lds, i64 rows, i64 cols, float scale,
                                                   __half* __restrict__ out, const int* __restrict__ skip_flag) {
  pdl_enter();
  if (skip_flag != nullptr && *skip_flag != 0) return;
  round_f16_body(src, lds, rows, cols, scale, out);
}
// (one launch over a chain: blockIdx.y, outputs `ostride` floats apart)
__global__ void __launch_bounds__(256) k_round_f16_chain(const ChainPtrs srcs, i64 lds, i64 rows, i64 cols, float scale,
                                                         __half* __restrict__ out, i64 ostride,
                                                         const int* __restrict__ skip_flag, i64 skip_stride) {
  pdl_enter();
  const i64 b = blockIdx.y;
  if (skip_flag != nullptr && skip_flag[b * skip_stride] != 0) return;
  round_f16_body(reinterpret_cast<const float*>(srcs.p[b]), lds, rows, cols, scale, out + 2 * b * ostride);
}

// ---- a panel as a pair of IEEE half arrays, scaled: 22 significant bits at the 16-bit MMA rate ----------------
// Half has 5 exponent bits, so the panel is scaled by a power of two that puts its largest entry in [2^13, 2^14):
// entries down to 2^-17 of the largest keep all 22 bits of the pair, smaller ones an absolute error of 2^-39 of
// the largest.  Two launches: per-block maxima of |x|, then the split (every block reduces the maxima again, in
// a fixed order; block 0 also writes 1 / scale^2, the factor that takes a Gram matrix of the pair back).
// blockIdx.y: the matrix of a chain (arrays `wstride` floats apart); skip flags a state slot apart.
constexpr int AMAX_PARTS = 512;
__global__ void __launch_bounds__(256) k_absmax_partial(const float* __restrict__ src, i64 ld, i64 rows, i64 cols,
                                                        float* __restrict__ part, i64 wstride, const int* __restrict__ skip_flag,
                                                        i64 skip_stride) {
  pdl_enter();
  if (skip_flag != nullptr && skip_flag[(i64)blockIdx.y * skip_stride] != 0) return;
  src += (i64)blockIdx.y * wstride; part += (i64)blockIdx.y * wstride;
  const i64 per_row = cols / 4, total = rows * per_row;
  float m = 0.f;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / per_row, c = (e - i * per_row) * 4;
    const float4 a = *reinterpret_cast<const float4*>(src + i * ld + c);
    m = fmaxf(fmaxf(m, fmaxf(fabsf(a.x), fabsf(a.y))), fmaxf(fabsf(a.z), fabsf(a.w)));
  }
  __shared__ float red[256];
  red[threadIdx.x] = m;
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {
    if ((int)threadIdx.x < w) red[threadIdx.x] = fmaxf(red[threadIdx.x], red[threadIdx.x + w]);
    __syncthreads();
  }
  if (threadIdx.x == 0) part[blockIdx.x] = red[0];
}
// other_inv < 0: the scalar written is 1 / scale^2 (both operands of the product are this array); else
// other_inv / scale (the other operand carries a fixed scale of its own), times *other_dev when that is given (the
// other operand's own 1 / scale, written by its split; blockIdx.y entries wstride apart like everything else).
__global__ void __launch_bounds__(256) k_split_f16_scaled(const float* __restrict__ src, i64 ld, i64 rows, i64 cols,
                                                          const float* __restrict__ part, int nparts,
                                                          __half* __restrict__ hi, __half* __restrict__ lo,
                                                          float* __restrict__ inv_scale2, i64 wstride,
                                                          const int* __restrict__ skip_flag, i64 skip_stride,
                                                          float other_inv, const float* __restrict__ other_dev = nullptr) {
  pdl_enter();
  if (skip_flag != nullptr && skip_flag[(i64)blockIdx.y * skip_stride] != 0) return;
  src += (i64)blockIdx.y * wstride; part += (i64)blockIdx.y * wstride; inv_scale2 += (i64)blockIdx.y * wstride;
  if (other_dev != nullptr) other_dev += (i64)blockIdx.y * wstride;
  hi += 2 * (i64)blockIdx.y * wstride; lo += 2 * (i64)blockIdx.y * wstride;
  __shared__ float red[256];
  float m = 0.f;
  for (int e = threadIdx.x; e < nparts; e += 256) m = fmaxf(m, part[e]);
  red[threadIdx.x] = m;
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {
    if ((int)threadIdx.x < w) red[threadIdx.x] = fmaxf(red[threadIdx.x], red[threadIdx.x + w]);
    __syncthreads();
  }
  const float amax = red[0];
  int ex = 14;                                   // amax = f 2^ex with f in [0.5, 1): scale 2^(14 - ex)
  if (amax > 0.f && amax < 3.0e38f) frexpf(amax, &ex);
  if (ex < -100) ex = -100;
  const float scale = ldexpf(1.f, 14 - ex);
  if (blockIdx.x == 0 && threadIdx.x == 0)
    *inv_scale2 = (other_inv < 0.f) ? ldexpf(1.f, 2 * (ex - 14))
                                    : other_inv * ldexpf(1.f, ex - 14) * (other_dev != nullptr ? *other_dev : 1.f);
  const i64 per_row = cols / 8, total = rows * per_row;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / per_row, c = (e - i * per_row) * 8;
    const float4 a = *reinterpret_cast<const float4*>(src + i * ld + c);
    const float4 b = *(reinterpret_cast<const float4*>(src + i * ld + c) + 1);
    const float v[8] = {scale * a.x, scale * a.y, scale * a.z, scale * a.w, scale * b.x, scale * b.y, scale * b.z, scale * b.w};
    __half h[8], l[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      h[q] = __float2half_rn(v[q]);
      l[q] = __float2half_rn(v[q] - __half2float(h[q]));
    }
    *reinterpret_cast<uint4*>(hi + i * cols + c) = *reinterpret_cast<const uint4*>(h);
    *reinterpret_cast<uint4*>(lo + i * cols + c) = *reinterpret_cast<const uint4*>(l);
  }
}

// hi = half(scale x), lo = half(scale x - hi) with a scale given by the caller (a power of two; for arrays whose
// entries are bounded, like the unit-norm columns of Q).  Sources from a pointer table (blockIdx.y), outputs
// `ostride` floats apart.
// ldo: leading dimension of the outputs (0: dense).
__global__ void __launch_bounds__(256) k_split_f16_fixed(const ChainPtrs srcs, i64 lds, i64 rows, i64 cols, float scale,
                                                         __half* __restrict__ hi, __half* __restrict__ lo, i64 ostride,
                                                         i64 ldo = 0, const int* __restrict__ skip_flag = nullptr,
                                                         i64 skip_stride = 0) {
  pdl_enter();
  const i64 bm = blockIdx.y;
  if (skip_flag != nullptr && skip_flag[bm * skip_stride] != 0) return;
  if (ldo == 0) ldo = cols;
  const float* __restrict__ src = reinterpret_cast<const float*>(srcs.p[bm]);
  hi += 2 * bm * ostride; lo += 2 * bm * ostride;
  const i64 per_row = cols / 8, total = rows * per_row;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 i = e / per_row, c = (e - i * per_row) * 8;
    const float4 a = *reinterpret_cast<const float4*>(src + i * lds + c);
    const float4 b = *(reinterpret_cast<const float4*>(src + i * lds + c) + 1);
    const float v[8] = {scale * a.x, scale * a.y, scale * a.z, scale * a.w, scale * b.x, scale * b.y, scale * b.z, scale * b.w};
    __half h[8], l[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      h[q] = __float2half_rn(v[q]);
      l[q] = __float2half_rn(v[q] - __half2float(h[q]));
    }
    *reinterpret_cast<uint4*>(hi + i * ldo + c) = *reinterpret_cast<const uint4*>(h);
    *reinterpret_cast<uint4*>(lo + i * ldo + c) = *reinterpret_cast<const uint4*>(l);
  }
}

}  // namespace dion

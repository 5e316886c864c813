// Tensor-core (tcgen05 / TMEM) engine of the large contractions, sm_100a only.
//
// One persistent, warp-specialised kernel computes C = op(A) * op(B) on 128 x BN
// output tiles:
//   warps 0-7   epilogue: TMEM -> registers -> fused epilogue -> global memory
//   warps 8-15  producers / converters (see the variants below)
//   warp  16    one elected thread issues tcgen05.mma and the commits
//   warp  17    (TMA variants) one elected thread issues the cp.async.bulk.tensor loads
// Accumulators are double buffered in TMEM (2 x BN columns), so the epilogue of a
// tile overlaps the main loop of the next one.  Every large operand is transformed on
// the way in: the momentum buffer is formed as M + G, and fp32 operands are split into
// a TF32 "hi" part and an fp32 "lo" remainder (3xTF32: hi*lo + lo*hi + hi*hi carries
// fp32 accuracy), or rounded to bf16 in the bf16-operand mode.  Variants:
//   TMA, fp32 mode (default): raw fp32 tiles land in the stage buffers by TMA; the
//     producer warps add and split in place.
//   TMA, bf16 operands from fp32 arrays: same loads; the producer warps add, round and
//     write bf16 operand tiles.
//   bf16 arrays (D16): TMA writes the operand tiles themselves; the producer warps join
//     the epilogue.
//   register path: the producer warps load global memory through registers (operands a
//     tensor map cannot describe).
// Coalesced epilogue (CE; the bf16-array variant and the fp32 TMA variant when there is no
// bf16 addend to stage): the epilogue warps pass their accumulator rows through shared-
// memory tiles and access global memory in whole row segments, 8 or 16 rows of the tile's
// full width per row quadrant at a time.  The plain epilogue (a lane writes its own row)
// remains for the other variants.
//
// Every wait on an mbarrier is bounded by a cycle budget: when it runs out the CTA
// marks itself dead, raises DION_STATUS_TIMEOUT and drains, so a protocol bug
// cannot hang the GPU.
#pragma once

#include <cuda.h>

#include "dion_common.cuh"
#include "simt_gemm.cuh"

namespace dion {
namespace umma {

constexpr int BM = 128;
constexpr int NUM_EPI_WARPS = 8;   // warp w: TMEM lanes 32 (w % 4) .., column half w / 4
constexpr int NUM_PROD_WARPS = 8;
constexpr int NUM_PROD_THREADS = NUM_PROD_WARPS * 32;
constexpr int NUM_THREADS = (NUM_EPI_WARPS + NUM_PROD_WARPS + 1) * 32;
constexpr int NUM_THREADS_TMA = NUM_THREADS + 32;   // one more warp issues the TMA loads
constexpr long long SPIN_LIMIT_CYCLES = 2000000000LL;  // about one second

struct Params {
  alignas(64) CUtensorMap tmA, tmA2, tmB, tmB2;   // TMA variants: tiles of A, of its addend (or its "lo" array), of B (and its "lo" array)
  GemmArgs g;
  int nM, nN;         // output tiles along M and N
  int splits;         // K splits (>= 1); partial sums go to g.part when > 1
  int kb_per_split;   // K blocks per split
  int nkb;            // K blocks in all
  int num_items;      // tiles * splits * matrices
  int raster_gw;      // > 0: rectangular outputs are walked in column panels of this many tile columns
  int items_per_matrix;   // tiles * splits; a batched launch (g.batch2 matrices, g.bs2 elements apart) walks matrix by matrix
  int kc;             // K blocks per accumulation chunk (see k_gemm_umma)
  int* status;        // device status word (DION_STATUS_TIMEOUT)
  long long spin_limit;   // cycle budget of every mbarrier wait (SPIN_LIMIT_CYCLES unless a test shortens it)
  int withhold_arrive;    // test hook of the register-path variant: the producer warps do not arrive for the first
                          // K block, so that the consumer's bounded wait runs out (no copy is in flight then)
  // batched launch whose outputs are the caller's arrays (g.c_tab / g.c2_tab given): per-matrix C and C2
  float* ctab[GEMM_TAB_MAX];
  const void* c2tab[GEMM_TAB_MAX];
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// 2-D tiled TMA load into this CTA's shared memory (no multicast); x is the innermost coordinate.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// 3-D tiled TMA load: z is the matrix of a batched launch (the fp32 operand maps are 3-D, extent 1 when not batched)
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
// The same for a CTA pair: the tile goes to THIS CTA's shared memory, the completion (complete_tx) to the mbarrier
// at cluster address `bar_cluster`, which may belong to either CTA of the pair (here: the leader's).  No multicast.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ uint32_t cluster_addr(uint32_t addr, uint32_t rank) {   // `addr` as seen in CTA `rank`
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 lds128(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, float4 v) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
// four floats rounded to bf16 (round to nearest even), stored as 8 bytes
__device__ __forceinline__ void sts64_bf16x4(uint32_t addr, float4 v) {
  const __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "r"(*reinterpret_cast<const uint32_t*>(&a)),
               "r"(*reinterpret_cast<const uint32_t*>(&b))
               : "memory");
}
// remainder of x after truncation to TF32 (what the MMA drops when it reads an fp32 word)
__device__ __forceinline__ float trunc_rem(float x) { return x - __uint_as_float(__float_as_uint(x) & 0xFFFFE000u); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---- CTA pair (cta_group::2): two CTAs of a cluster share one 256-row MMA
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on the mbarrier at the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar, uint32_t rank) {
  asm volatile(
      "{\n\t.reg .b32 ra;\n\t"
      "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
      "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n\t}" ::"r"(bar), "r"(rank)
      : "memory");
}
// The same without release semantics: for an arrival that orders nothing but tcgen05 operations (which
// tcgen05.fence::before_thread_sync orders).  A release at cluster scope makes the thread wait until its earlier
// global stores are visible cluster-wide: a memory round trip per tile for an epilogue warp.
__device__ __forceinline__ void mbar_arrive_remote_relaxed(uint32_t bar, uint32_t rank) {
  asm volatile(
      "{\n\t.reg .b32 ra;\n\t"
      "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
      "mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [ra];\n\t}" ::"r"(bar), "r"(rank)
      : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tmem_alloc2(uint32_t slot, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// one 256 x N x 8 TF32 MMA of the CTA pair, issued by the leader CTA
__device__ __forceinline__ void umma2_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the same with bf16 operands (256 x N x 16)
__device__ __forceinline__ void umma2_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// commit of the pair's MMAs: arrives on the mbarrier at this offset in every CTA of `mask`
__device__ __forceinline__ void umma2_commit(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"(mask)
               : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t slot, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
template <bool BF16>
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  if (BF16) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
template <bool WAIT = true>
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  if (WAIT) asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// 16 columns of the lane's row
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t cvt_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Bounded wait: false when the CTA is (or becomes) dead.
// `sleep_ns` > 0 backs off between polls so that a waiting warp does not take issue
// slots from the producer warps.
template <bool CLUSTER = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* dead, int* status,
                                          long long limit, unsigned sleep_ns = 0) {
  // CLUSTER: the barrier takes arrivals from the peer CTA (acquire at cluster scope)
  if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  unsigned polls = 0;
  while (true) {
    if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if (sleep_ns) __nanosleep(sleep_ns);
    if ((++polls & 63u) == 0) {
      if (*dead) return false;
      if (clock64() - t0 > limit) {
        *dead = 1;
        atomicOr(status, DION_STATUS_TIMEOUT);
        return false;
      }
    }
  }
}

// Shared-memory matrix descriptor.
// K-major (any type) and MN-major bf16: 128-byte swizzle (16-byte units XORed with
//   the row index mod 8); rows of 128 bytes, 8-row groups 1024 bytes apart.
// MN-major TF32: the only layout the hardware takes is the 128-byte swizzle with a
//   32-byte base: atoms of 4 k-rows x 128 bytes, 32-byte units XORed with the row
//   index mod 4; groups of 4 k-rows are 512 bytes apart.
// For MN-major operands `lbo_bytes` is the distance between consecutive 128-byte
// chunks along M/N (32 fp32 or 64 bf16 elements).
template <bool BF16>
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, bool mn_major, uint32_t lbo_bytes) {
  const bool base32 = mn_major && !BF16;
  const uint64_t lbo = mn_major ? (uint64_t)(lbo_bytes >> 4) : 1ull;
  const uint64_t sbo = base32 ? (512 >> 4) : (1024 >> 4);
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= lbo << 16;
  d |= sbo << 32;
  d |= 1ull << 46;                      // descriptor version of sm_100
  d |= (base32 ? 1ull : 2ull) << 61;    // SWIZZLE_128B_BASE32B or SWIZZLE_128B
  return d;
}

// k-contiguous bf16 tile with rows of 64 bytes (32 elements): 64-byte swizzle (16-byte
// units XORed with bits 1-2 of the row index), 8-row groups 512 bytes apart.
__device__ __forceinline__ uint64_t make_desc_k64(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= 1ull << 16;
  d |= (uint64_t)(512 >> 4) << 32;
  d |= 1ull << 46;
  d |= 4ull << 61;                      // SWIZZLE_64B
  return d;
}

// Instruction descriptor: fp32 accumulate, TF32 or BF16 operands, M = 128, N = BN.
// f16 (with bf16): the 16-bit operands are IEEE half values (kind::f16 takes either format)
__device__ __forceinline__ uint32_t make_idesc(bool bf16, bool a_mn, bool b_mn, int bn, int bm = BM, bool f16 = false) {
  uint32_t d = 0;
  const uint32_t fmt = bf16 ? (f16 ? 0u : 1u) : 2u;   // 0 F16, 1 BF16 (kind::f16); 2 TF32 (kind::tf32)
  d |= 1u << 4;                         // D format: F32
  d |= fmt << 7;                        // A format
  d |= fmt << 10;                       // B format
  d |= (a_mn ? 1u : 0u) << 15;
  d |= (b_mn ? 1u : 0u) << 16;
  d |= (uint32_t)(bn >> 3) << 17;
  d |= (uint32_t)(bm >> 4) << 24;
  return d;
}

constexpr i64 TRI_WIDE_MIN = 4096;   // smallest lower-triangular output computed in 128 x 256 tiles

struct Item {
  int mi, ni, ks, kb0, kb1;
  int b;      // matrix of a batched launch
};

// CG2: `mi` counts 256-row tiles of a CTA pair (256 x 256 lower tiles in the triangular case).
template <int BN, int BKE, bool CG2 = false>
__device__ __forceinline__ Item decode_item(const Params& p, int item) {
  Item it;
  it.b = item / p.items_per_matrix;
  item -= it.b * p.items_per_matrix;
  const int tile = item / p.splits;
  it.ks = item - tile * p.splits;
  if (p.g.tri == TRI_LOWER && BN == 2 * BM && !CG2) {
    // 128 x 256 tiles that reach the diagonal or lie below it: tile row mi has mi / 2 + 1 of them,
    // (mi + 1)^2 / 4 (rounded down) lie in the rows above it
    int mi = (int)(2.f * sqrtf((float)tile)) - 1;
    if (mi < 0) mi = 0;
    while ((mi + 2) * (mi + 2) / 4 <= tile) ++mi;
    while ((mi + 1) * (mi + 1) / 4 > tile) --mi;
    it.mi = mi;
    it.ni = tile - (mi + 1) * (mi + 1) / 4;
  } else if (p.g.tri == TRI_LOWER) {
    int mi = (int)((sqrtf(8.f * (float)tile + 1.f) - 1.f) * 0.5f);
    while ((mi + 1) * (mi + 2) / 2 <= tile) ++mi;
    while (mi * (mi + 1) / 2 > tile) --mi;
    it.mi = mi;
    it.ni = tile - mi * (mi + 1) / 2;
  } else if (p.raster_gw > 0) {
    // column panels of raster_gw tile columns, walked row by row: the tiles in flight share the panel's B blocks
    // (which stay in L2 for the whole panel) instead of sweeping all of B once per wave
    const int per_panel = p.nM * p.raster_gw;
    const int pn = tile / per_panel;
    const int rem = tile - pn * per_panel;
    const int n0 = pn * p.raster_gw;
    const int gw = min(p.raster_gw, p.nN - n0);
    it.mi = rem / gw;
    it.ni = n0 + (rem - it.mi * gw);
  } else {
    it.mi = tile / p.nN;
    it.ni = tile - it.mi * p.nN;
  }
  int nkb = p.nkb;
  if (p.g.klimit) {
    const i64 kend = min(p.g.K, (i64)(it.ni + 1) * BN);
    nkb = (int)((kend + BKE - 1) / BKE);
  }
  it.kb0 = it.ks * p.kb_per_split;
  it.kb1 = min(nkb, it.kb0 + p.kb_per_split);
  return it;
}

// Where the 16-byte chunks of one producer thread sit, computed once per kernel:
// an operand tile is ROWS x BKE elements and is cut into chunks of EPC elements.
// MN_MAJOR = false: memory is contiguous along k (chunk = EPC consecutive k of one
// row); true: contiguous along the row index (chunk = EPC consecutive rows at one k).
//   goff  element offset of the chunk from the tile's (row0, k0) corner in memory
//   soff  byte offset of the chunk in the stage buffer (swizzled canonical layout)
//   rpos / kpos  first row / k of the chunk inside the tile (for the edge predicates)
template <int ROWS, int BKE, int EPC, bool MN_MAJOR, int NCHUNK, bool BF16>
struct TileMap {
  uint32_t goff[NCHUNK];
  uint32_t goff2[NCHUNK];
  uint32_t soff[NCHUNK];   // bits 0-19 offset, 20-25 kpos, 26-31 unused
  uint16_t rpos[NCHUNK];

  __device__ __forceinline__ void init(int ptid, i64 s_row, i64 s_k, i64 s2_row, i64 s2_k) {
    constexpr int CPR = MN_MAJOR ? (ROWS / EPC) : (BKE / EPC);   // chunks per k-row / per row
#pragma unroll
    for (int l = 0; l < NCHUNK; ++l) {
      const int c = ptid + l * NUM_PROD_THREADS;
      const int major = c / CPR, minor = c % CPR;
      const int row = MN_MAJOR ? minor * EPC : major;
      const int kk = MN_MAJOR ? major : minor * EPC;
      goff[l] = (uint32_t)(row * s_row + kk * s_k);
      goff2[l] = (uint32_t)(row * s2_row + kk * s2_k);
      rpos[l] = (uint16_t)row;
      uint32_t off;
      if (MN_MAJOR && !BF16) {   // TF32, row-contiguous: 32-byte swizzle units, atoms of 4 k-rows
        const uint32_t q = (uint32_t)(minor & 7);
        off = (uint32_t)(minor >> 3) * (BKE * 128) + (uint32_t)major * 128 + ((((q >> 1) ^ (uint32_t)(major & 3))) << 5) +
              ((q & 1u) << 4);
      } else if (MN_MAJOR) {     // bf16, row-contiguous
        off = (uint32_t)(minor >> 3) * (BKE * 128) + (uint32_t)major * 128 + (uint32_t)(((minor & 7) ^ (major & 7)) << 4);
      } else {                   // k-contiguous: rows of 128 bytes, 16-byte units XOR (row mod 8)
        off = (uint32_t)major * 128 + (uint32_t)((minor ^ (major & 7)) << 4);
      }
      soff[l] = off | ((uint32_t)kk << 20);
    }
  }

  // Loads the tile whose corner is at `src` (and `src2` for the fused addend).  `rows_left`
  // / `k_left`: how many rows / k remain from the corner (edge tiles are zero filled).
  // All loads are issued before any value is used, so their latencies overlap; the
  // addend is kept raw in `w` (fp32 values, or packed bf16 pairs) until add() runs.
  __device__ __forceinline__ void load(const float* __restrict__ src, const void* __restrict__ src2, int add_mode,
                                       i64 rows_left, i64 k_left, float (&v)[NCHUNK][EPC], float (&w)[NCHUNK][EPC]) const {
    const bool interior = rows_left >= ROWS && k_left >= BKE;
#pragma unroll
    for (int l = 0; l < NCHUNK; ++l) {
      const bool ok = interior || ((i64)rpos[l] < rows_left && (i64)(soff[l] >> 20) < k_left);
#pragma unroll
      for (int q = 0; q < EPC / 4; ++q) {
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ok) t = __ldg(reinterpret_cast<const float4*>(src + goff[l]) + q);
        v[l][q * 4 + 0] = t.x; v[l][q * 4 + 1] = t.y; v[l][q * 4 + 2] = t.z; v[l][q * 4 + 3] = t.w;
      }
      if (add_mode == ADD_F32) {
#pragma unroll
        for (int q = 0; q < EPC / 4; ++q) {
          float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
          if (ok) t = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(src2) + goff2[l]) + q);
          w[l][q * 4 + 0] = t.x; w[l][q * 4 + 1] = t.y; w[l][q * 4 + 2] = t.z; w[l][q * 4 + 3] = t.w;
        }
      } else if (add_mode == ADD_BF16) {
#pragma unroll
        for (int q = 0; q < EPC / 4; ++q) {
          uint2 t = make_uint2(0u, 0u);
          if (ok) t = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(src2) + goff2[l]) + q);
          w[l][q * 4 + 0] = __uint_as_float(t.x); w[l][q * 4 + 1] = __uint_as_float(t.y);
        }
      }
    }
  }

  // v += addend (after load()).
  __device__ __forceinline__ void add(int add_mode, float (&v)[NCHUNK][EPC], const float (&w)[NCHUNK][EPC]) const {
    if (add_mode == ADD_F32) {
#pragma unroll
      for (int l = 0; l < NCHUNK; ++l)
#pragma unroll
        for (int e = 0; e < EPC; ++e) v[l][e] += w[l][e];
    } else if (add_mode == ADD_BF16) {
#pragma unroll
      for (int l = 0; l < NCHUNK; ++l)
#pragma unroll
        for (int q = 0; q < EPC / 4; ++q) {
          const uint32_t x = __float_as_uint(w[l][q * 4 + 0]), y = __float_as_uint(w[l][q * 4 + 1]);
          const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&x);
          const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&y);
          v[l][q * 4 + 0] += __low2float(lo); v[l][q * 4 + 1] += __high2float(lo);
          v[l][q * 4 + 2] += __low2float(hi); v[l][q * 4 + 3] += __high2float(hi);
        }
    }
  }

  // Writes the chunks to shared memory.  fp32 mode: TF32 "hi" part to s_hi and the TF32-
  // rounded remainder to s_lo; bf16 mode: rounded to bf16 into s_hi.
  __device__ __forceinline__ void store(uint32_t s_hi, uint32_t s_lo, const float (&v)[NCHUNK][EPC]) const {
#pragma unroll
    for (int l = 0; l < NCHUNK; ++l) {
      const uint32_t off = soff[l] & 0xFFFFFu;
      if (BF16) {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const __nv_bfloat162 b = __floats2bfloat162_rn(v[l][q * 2], v[l][q * 2 + 1]);
          w[q] = *reinterpret_cast<const uint32_t*>(&b);
        }
        st_shared_v4(s_hi + off, w[0], w[1], w[2], w[3]);
      } else {
        uint32_t h[4], lo[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          h[q] = cvt_tf32(v[l][q]);
          lo[q] = __float_as_uint(v[l][q] - __uint_as_float(h[q]));
        }
        st_shared_v4(s_hi + off, h[0], h[1], h[2], h[3]);
        st_shared_v4(s_lo + off, lo[0], lo[1], lo[2], lo[3]);
      }
    }
  }
};

// SPLIT (fp32 mode only): the hi*hi products and the small hi*lo + lo*hi products go
// to separate TMEM accumulators that are added once in the epilogue.  Every
// tcgen05.mma truncates when it adds into its accumulator; keeping the small terms
// apart leaves one such truncation per K step on the main sum instead of three and
// brings the product to the accuracy of an fp32 FMA loop (measured 3.3e-7 against
// 9.1e-7 relative error on Gaussian data).  Used for the products whose error the
// conditioning of an ill-conditioned panel amplifies.
// ONE (fp32 mode, single pass): the operands are fp32 arrays whose values already fit TF32 (rounded to
// nearest beforehand, k_round_tf32), so one kind::tf32 MMA per K step reads the raw tiles TMA has written:
// no "lo" halves, no conversion pass, the producer warps join the epilogue as in the bf16-array variant.
// Used for the rank-r update of X, whose result feeds nothing else: an unbiased 2^-12 relative operand
// error there moves X by ~1e-6.
// CG2 (TMA, BN = 256): two CTAs of a cluster form one 256 x 256 tile with cta_group::2 MMAs.
// Each CTA loads and converts its own 128 rows of A and HALF of the B tile (128 of the 256 columns), so a
// K block costs a CTA two thirds of the shared-memory traffic of the single-CTA form (which is bound by
// it: three MMAs re-read both operand tiles) and a stage is 64 KB instead of 96 KB (3 stages instead of 2).
// The leader CTA issues the MMAs for both; accumulators and epilogue stay per CTA (128 rows x 256 columns).
// The variants on 16-bit arrays (D16: nothing to convert) form pairs too: both CTAs' TMA loads then complete on the
// leader's barrier (cta_group::2 load form), which the leader's MMA thread waits on.
// X2 (bf16 arrays, D16): each operand is a PAIR of bf16 arrays, x ~ hi + lo with hi = bf16(x), lo = bf16(x - hi)
// (16 significant bits); three bf16 MMAs per K step (hi*lo + lo*hi + hi*hi) give a product that is accurate to
// ~1e-5 relative at 1.3 times the tensor time of one TF32 pass.  Used for the error-feedback product in fp32
// mode, whose result enters M scaled by 1 - mu.
template <int BN, bool BF16, bool SPLIT = false, bool TMA = false, bool D16 = false, bool CE = false, bool ONE = false,
          bool CG2 = false, bool X2 = false>
struct Cfg {
  // BT: bf16 operands formed in shared memory from TMA-loaded fp32 tiles (K block of 32, as in
  // the fp32 TMA variant).  A stage then holds the raw fp32 tiles of A, of its fp32 addend and
  // of B, followed by the bf16 operand tiles of A and B (half the bytes each).
  // D16: both operands are bf16 arrays in memory; TMA writes the operand tiles themselves
  // (K block of 64, 128-byte swizzle) and the producer warps have nothing to do.
  static constexpr bool BT = BF16 && TMA && !D16;
  static constexpr int BKE = (BF16 && (!TMA || D16)) ? 64 : 32;   // K elements per stage
  static constexpr int EPC = (BF16 && !TMA) ? 8 : 4;         // elements per 16-byte chunk of the register path
  static constexpr int A_BYTES = BM * 128;
  static constexpr int BN_L = CG2 ? BN / 2 : BN;             // columns of the B tile this CTA holds
  static constexpr int B_BYTES = BN_L * 128;
  static constexpr int STAGE_BYTES = BT ? (2 * A_BYTES + B_BYTES + A_BYTES / 2 + B_BYTES / 2)
                                        : (((BF16 && !X2) || ONE) ? 1 : 2) * (A_BYTES + B_BYTES);
  // D16: the producer warps have no conversion work and serve as epilogue warps too
  // (with operand pairs the stages leave room for 8 warps' epilogue tiles only)
  static constexpr int EPI_WARPS = ((D16 && !X2) || ONE) ? NUM_EPI_WARPS + NUM_PROD_WARPS : NUM_EPI_WARPS;
  // Operand pairs: nothing to convert and no room for more epilogue tiles, so the kernel runs without the producer
  // warps (10 warps in all); the registers they would hold go to the epilogue warps' loads in flight (DEEP).
  static constexpr bool DEEP = X2;
  static constexpr int MMA_WARP = X2 ? NUM_EPI_WARPS : NUM_EPI_WARPS + NUM_PROD_WARPS;   // the warp that issues the MMAs
  static constexpr int THREADS = (MMA_WARP + (TMA ? 2 : 1)) * 32;                         // ... then the TMA warp
  // CE (coalesced epilogue): an epilogue warp owns 32 rows x EPI_W columns of the tile and passes them
  // through a private shared-memory tile in passes of EPI_RPP rows (EPI_RPP * EPI_W = 1024 elements),
  // so that one global access of the warp covers whole row segments instead of 32 rows; paid for with
  // a pipeline stage (bf16 arrays) or the addend staging (fp32 operands: the products that use this
  // epilogue have no fused addend).
  static constexpr int EPI_W = 32 * (BN / 32) / (EPI_WARPS / 4);
  static constexpr int EPI_RPP = 1024 / EPI_W;
  static constexpr int EPI_TILE_FLOATS = EPI_RPP * (EPI_W + 4);
  static constexpr int EPI_BYTES = CE ? EPI_WARPS * EPI_TILE_FLOATS * 4 : 0;
  static constexpr int STAGES = CE ? (232448 - 1536 - EPI_BYTES) / STAGE_BYTES : (192 * 1024) / STAGE_BYTES;
  static constexpr int G16_BYTES = ((BF16 && !TMA) || D16 || CE) ? 0 : BM * 32 * 2;   // bf16 addend tile of the TMA variants (per stage)
  static constexpr int SMEM_BYTES = STAGES * (STAGE_BYTES + G16_BYTES) + EPI_BYTES + 1024 + 512;
  static constexpr int A_CHUNKS = BM * 8 / NUM_PROD_THREADS;  // 16-byte chunks per producer thread
  static constexpr int B_CHUNKS = BN_L * 8 / NUM_PROD_THREADS;
  static constexpr int ACCS = SPLIT ? 2 : 1;                 // accumulators per tile
  static constexpr int NBUF = (512 / (ACCS * BN)) >= 2 ? 2 : 1;  // tiles in flight in TMEM
  static constexpr int TMEM_COLS = NBUF * ACCS * BN;
  static constexpr int KSTEPS = BT ? 2 : 4;                  // UMMA K steps per stage
};

// TMA = true: a dedicated warp loads the raw fp32 tiles of A, of its addend and
// of B with TMA straight into the stage buffers (A and B into their "hi" halves, the
// addend into A's "lo" half).  The 8 producer warps then only convert in place: the MMA
// truncates an fp32 word to TF32 by itself, so the raw word serves as the "hi" operand
// and only the truncation remainder is written to the "lo" half (after the M + G add
// for a fused A).  Loads of one stage overlap conversion and MMAs of the other, and
// out-of-range rows / k are zero filled by the TMA unit.
// TMA with bf16 operands: the same loads; the producer warps add, round to bf16 and write
// the operand tiles the MMA reads (k-contiguous: rows of 64 bytes, 64-byte swizzle;
// row-contiguous: 128-byte rows of 64 row indices, 128-byte swizzle); one MMA per K step.
template <int BN, bool A_MN, bool B_MN, bool BF16, bool SPLIT, bool TMA, bool D16 = false, bool CE = false, bool ONE = false,
          bool CG2 = false, bool X2 = false>
__global__ void __launch_bounds__((Cfg<BN, BF16, SPLIT, TMA, D16, CE, ONE, CG2, X2>::THREADS), 1)
k_gemm_umma(const __grid_constant__ Params p) {
  static_assert(!X2 || (D16 && CE), "operand pairs are bf16 arrays");
  static_assert(!CG2 || (TMA && BN == 256 && ((!BF16 && !D16 && !ONE) || (D16 && CE))),
                "CTA pairs: the fp32 TMA variants and the 16-bit array variants (single arrays or pairs), 256-column tiles");
  static_assert(!(BF16 && SPLIT) || X2, "split accumulators belong to the 3xTF32 mode and to operand pairs");
  static_assert(!D16 || (BF16 && TMA), "bf16 operands in memory are loaded by TMA");
  static_assert(!CE || (TMA && (D16 || !BF16)), "the coalesced epilogue serves the bf16-array and the fp32 TMA variants");
  static_assert(!ONE || (TMA && CE && !BF16 && !SPLIT && !A_MN && !B_MN), "single pass: k-contiguous fp32 operands by TMA");
  using C = Cfg<BN, BF16, SPLIT, TMA, D16, CE, ONE, CG2, X2>;
  constexpr bool NOCONV = D16 || ONE;    // the operand tiles are what TMA writes: nothing to convert
  constexpr bool PAIRLOAD = CG2 && NOCONV;   // both CTAs' loads complete on the leader's barrier
  constexpr int BN_L = C::BN_L;
  const uint32_t cta_rank = CG2 ? cluster_ctarank() : 0u;   // 0: the leader of the pair
  const int worker = CG2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;       // which tile stream this CTA (pair) walks
  const int workers = CG2 ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  constexpr int NBUF = C::NBUF, ACCS = C::ACCS;
  constexpr int BKE = C::BKE, EPC = C::EPC, STAGES = C::STAGES;
  // a launch over one matrix does nothing when that matrix's flag is set; a batched launch skips flagged matrices
  // item by item (every role reads the same flags, which no kernel writes while this one runs)
  const bool batched = p.g.batch2 > 1;
  if (!batched && p.g.skip_flag != nullptr && *p.g.skip_flag != 0) return;
  auto skipped = [&](const Item& it) -> bool {
    return batched && p.g.skip_flag != nullptr && p.g.skip_flag[(i64)it.b * p.g.skip_stride] != 0;
  };

  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
  // control block after the stages
  // after the stages: the bf16 addend staging of the TMA variant, then the control block
  const uint32_t g16_base = smem_base + STAGES * C::STAGE_BYTES;
  float* epi_tiles = reinterpret_cast<float*>(smem_al + STAGES * (C::STAGE_BYTES + C::G16_BYTES));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * (C::STAGE_BYTES + C::G16_BYTES) + C::EPI_BYTES);
  const uint32_t bar0 = smem_base + STAGES * (C::STAGE_BYTES + C::G16_BYTES) + C::EPI_BYTES;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
  const uint32_t drain_bar = bar0 + 8u * (2 * STAGES + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 2 * STAGES + 5);
  volatile int* dead = reinterpret_cast<volatile int*>(bars + 2 * STAGES + 6);
  auto raw_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 7 + s); };   // TMA landed (TMA variant)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    // CTA pair: the leader's "full" and "accumulator free" barriers take the arrivals of both CTAs
    // (nothing to convert: "full" is unused then)
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), NOCONV ? 1 : NUM_PROD_WARPS * (CG2 ? 2 : 1)); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(accf_bar(b), 1); mbar_init(acce_bar(b), C::EPI_WARPS * (CG2 ? 2 : 1)); }   // one arrival per epilogue warp
    mbar_init(drain_bar, 1);
    // (pair without converters: the leader's "landed" barrier counts the bytes of both CTAs' tiles, see the TMA issuer)
    if (TMA) for (int s = 0; s < STAGES; ++s) mbar_init(raw_bar(s), 1);
    *dead = 0;
    fence_barrier_init();
  }
  if (warp == C::MMA_WARP) {
    if (CG2) { tmem_alloc2(smem_u32((const void*)tmem_slot), C::TMEM_COLS); tmem_relinquish2(); }
    else { tmem_alloc(smem_u32((const void*)tmem_slot), C::TMEM_COLS); tmem_relinquish(); }
  }
  tc_fence_before();
  __syncthreads();
  if (CG2) cluster_sync_all();      // the peer's barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const GemmArgs& g = p.g;

  if (warp < C::EPI_WARPS) {
    // ------------------------------------------------------------ epilogue
    // The tensor core adds into its accumulator with truncation, so the error of a long
    // accumulation chain grows linearly with its length (measured 7e-9 per k element).
    // The K loop of a tile is therefore cut into chunks of p.kc K blocks; each chunk is
    // accumulated from zero in TMEM and added here, in fp32 round-to-nearest, to the
    // running result in global memory.
    int iter = 0;
    bool alive = true;
    for (int item = worker; item < p.num_items && alive; item += workers) {
      Item it = decode_item<BN, BKE, CG2>(p, item);
      if (skipped(it)) continue;
      if (CG2) it.mi = 2 * it.mi + (int)cta_rank;     // this CTA's 128 rows of the pair's tile
      float* const Cb = (g.c_tab != nullptr) ? p.ctab[it.b] : g.C + (i64)it.b * g.bs2;   // this matrix's output ...
      float* const partb = g.part + (i64)it.b * g.bs2;                             // ... split-K partial sums ...
      const void* const C2b = (g.c2_tab != nullptr) ? p.c2tab[it.b]                // ... and second epilogue operand
                              : (g.c2_batched && g.C2 != nullptr)                  //     (fp32, in scratch)
                                  ? (const void*)(reinterpret_cast<const float*>(g.C2) + (i64)it.b * g.bs2) : g.C2;
      const int quad = warp & 3, half = warp >> 2;   // TMEM lane quadrant, column part
      constexpr int SLABS = (BN / 32) / (C::EPI_WARPS / 4);   // 32-column slabs per warp
      const i64 gi = (i64)it.mi * BM + quad * 32 + lane;
      const i64 n0 = (i64)it.ni * BN;
      // (a device scalar: the learning rate under graph replay, or a matrix's own scale)
      const float alpha = g.alpha * (g.alpha_dev != nullptr ? __ldg(g.alpha_dev + (i64)it.b * g.alpha_dev_stride) : 1.f);
      for (int kb = it.kb0; kb < it.kb1; kb += p.kc, ++iter) {
        const bool first = (kb == it.kb0);
        const int ab = iter % NBUF;
        const uint32_t ph = (uint32_t)(iter / NBUF) & 1u;
        if constexpr (CE) {
          // Coalesced epilogue.  A TMEM lane is a row, so a warp that wrote its accumulator rows straight
          // out would touch 32 rows per global access.  Instead the warp handles its 32 rows x W columns
          // (W = 32 SLABS) in passes of RPP rows: it reads its slabs from TMEM, the lanes of the pass's
          // rows put theirs into the warp's shared-memory tile, and the warp then accesses memory row
          // by row (an instruction covers RPI rows of W contiguous columns).  The warps of a row
          // quadrant own neighbouring column ranges, so a quadrant pass reads and writes RPP full row
          // segments of the tile (BN columns: 1 KB at BN = 256) at about the same time; that locality
          // is worth 25-30 % of DRAM bandwidth against 32 x 32 slabs handled one after another.
          constexpr int W = C::EPI_W;
          constexpr int RPP = C::EPI_RPP;     // rows per pass
          constexpr int LPR = W / 4;          // lanes per row
          constexpr int RPI = 32 / LPR;       // rows per instruction
          constexpr int NI = RPP / RPI;       // instructions per pass (8)
          constexpr int TS = W + 4;           // tile row stride (floats)
          constexpr int NP = 32 / RPP;        // passes
          static_assert(W == 32 * SLABS && NI == 8, "pass geometry");
          float* tb = epi_tiles + warp * C::EPI_TILE_FLOATS;
          const bool to_part = p.splits > 1;
          const bool need_c = !first || (!to_part && g.epi != EPI_STORE && g.epi != EPI_C2_SUB);
          const bool add_c2 = !to_part && first && (g.epi == EPI_ADD2_SUB || g.epi == EPI_C2_SUB);
          const bool c2_f32 = (g.c2_mode == ADD_F32 || g.epi == EPI_C2_SUB);
          const i64 col = n0 + half * W + 4 * (lane % LPR);
          float f = 1.f;
          if (!to_part) f = (g.epi != EPI_STORE) ? -alpha : alpha;
          // rows of pass ps that this lane touches: row0 + ps * RPP + RPI * q
          const i64 row0 = (i64)it.mi * BM + quad * 32 + lane / LPR;
          auto out_ptr = [&](i64 row) -> float4* {
            return to_part ? reinterpret_cast<float4*>(partb + ((i64)it.ks * g.M + row) * g.N + col)
                           : reinterpret_cast<float4*>(Cb + row * g.ldc + col);
          };
          auto c2_load = [&](i64 row) -> float4 {
            if (c2_f32) return __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(C2b) + row * g.ldc2 + col));
            const uint2 t = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(C2b) + row * g.ldc2 + col));
            const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&t.x);
            const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&t.y);
            return make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
          };
          // What the accumulator is added to (the running C, the second operand, or both) does not depend on the
          // MMAs: the loads of a pass are issued before its rows are read from TMEM and staged (those of the first
          // pass before the wait for the accumulator) and meet them only in `combine`, so that their latency is
          // covered by that work.
          auto fetch = [&](int ps, float4 (&buf)[NI]) {
#pragma unroll
            for (int q = 0; q < NI; ++q) {
              const i64 row = row0 + ps * RPP + RPI * q;
              float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
              if (row < g.M && col < g.N) {
                if (need_c && add_c2) {
                  const float4 c = *out_ptr(row);
                  const float4 t = c2_load(row);
                  v = make_float4(c.x + t.x, c.y + t.y, c.z + t.z, c.w + t.w);
                } else if (need_c) {
                  v = *out_ptr(row);
                } else if (add_c2) {
                  v = c2_load(row);
                }
              }
              buf[q] = v;
            }
          };
          auto stage_rows = [&](int ps) {     // rows ps * RPP .. of the warp's 32, from TMEM into the warp's tile
            // 16 columns at a time where the loads in flight need the registers (8 epilogue warps: wide passes)
            constexpr int LDW = (C::EPI_WARPS > 8) ? 32 : 16;
#pragma unroll
            for (int sl = 0; sl < W / LDW; ++sl) {
              float acc[LDW];
              const uint32_t ta = tmem_base + (uint32_t)(ab * ACCS * BN + half * W + sl * LDW) + ((uint32_t)(quad * 32) << 16);
              if constexpr (LDW == 32) tmem_ld32(ta, acc);
              else tmem_ld16(ta, acc);
              if (SPLIT) {
                float small[LDW];
                if constexpr (LDW == 32) tmem_ld32(ta + (uint32_t)BN, small);
                else tmem_ld16(ta + (uint32_t)BN, small);
#pragma unroll
                for (int e = 0; e < LDW; ++e) acc[e] += small[e];
              }
              if (lane / RPP == ps) {
#pragma unroll
                for (int q = 0; q < LDW / 4; ++q)
                  *reinterpret_cast<float4*>(tb + (lane % RPP) * TS + sl * LDW + 4 * q) =
                      make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]);
              }
            }
          };
          auto combine = [&](int ps, const float4 (&buf)[NI]) {
#pragma unroll
            for (int q = 0; q < NI; ++q) {
              const i64 row = row0 + ps * RPP + RPI * q;
              if (!(row < g.M && col < g.N)) continue;
              const float4 a4 = *reinterpret_cast<const float4*>(tb + (RPI * q + lane / LPR) * TS + 4 * (lane % LPR));
              const float4 c = buf[q];
              *out_ptr(row) = make_float4(fmaf(f, a4.x, c.x), fmaf(f, a4.y, c.y), fmaf(f, a4.z, c.z), fmaf(f, a4.w, c.w));
            }
          };
          auto release = [&]() {     // the accumulator has been read: the next tile's MMAs may overwrite it
            tc_fence_before();
            __syncwarp();          // every lane's TMEM reads are done; one (possibly remote) arrival per warp
            if (lane == 0) {
              if (CG2 && cta_rank != 0) mbar_arrive_remote_relaxed(acce_bar(ab), 0u);
              else mbar_arrive(acce_bar(ab));
            }
          };
          if constexpr (SPLIT) {
            // two accumulators to read per slab: no registers to spare for loads in flight across the staging
            if (!mbar_wait(accf_bar(ab), ph, dead, p.status, p.spin_limit, 256)) { alive = false; break; }
            tc_fence_after();
            float4 b0[NI];
#pragma unroll 1
            for (int ps = 0; ps < NP; ++ps) {
              stage_rows(ps);
              __syncwarp();
              if (ps + 1 == NP) release();
              fetch(ps, b0);
              combine(ps, b0);
              __syncwarp();      // the tile is rewritten by the next pass
            }
          } else if constexpr (C::DEEP) {
            // registers to spare: C and the second operand wait in registers of their own (no arithmetic, hence
            // no wait, at issue time)
            auto fetch2 = [&](int ps, float4 (&bc)[NI], float4 (&bt)[NI]) {
#pragma unroll
              for (int q = 0; q < NI; ++q) {
                const i64 row = row0 + ps * RPP + RPI * q;
                const bool ok = row < g.M && col < g.N;
                bc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                bt[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (ok && need_c) bc[q] = *out_ptr(row);
                if (ok && add_c2) bt[q] = c2_load(row);
              }
            };
            auto combine2 = [&](int ps, const float4 (&bc)[NI], const float4 (&bt)[NI]) {
#pragma unroll
              for (int q = 0; q < NI; ++q) {
                const i64 row = row0 + ps * RPP + RPI * q;
                if (!(row < g.M && col < g.N)) continue;
                const float4 a4 = *reinterpret_cast<const float4*>(tb + (RPI * q + lane / LPR) * TS + 4 * (lane % LPR));
                const float4 c = make_float4(bc[q].x + bt[q].x, bc[q].y + bt[q].y, bc[q].z + bt[q].z, bc[q].w + bt[q].w);
                *out_ptr(row) = make_float4(fmaf(f, a4.x, c.x), fmaf(f, a4.y, c.y), fmaf(f, a4.z, c.z), fmaf(f, a4.w, c.w));
              }
            };
            float4 c0[NI], t0[NI];
            fetch2(0, c0, t0);
            if (!mbar_wait(accf_bar(ab), ph, dead, p.status, p.spin_limit, 256)) { alive = false; break; }
            tc_fence_after();
#pragma unroll 1
            for (int ps = 0; ps < NP; ++ps) {
              stage_rows(ps);
              __syncwarp();
              if (ps + 1 == NP) release();
              combine2(ps, c0, t0);
              __syncwarp();      // the tile is rewritten by the next pass
              if (ps + 1 < NP) fetch2(ps + 1, c0, t0);
            }
          } else {
            float4 b0[NI];
            fetch(0, b0);
            if (!mbar_wait(accf_bar(ab), ph, dead, p.status, p.spin_limit, 256)) { alive = false; break; }
            tc_fence_after();
#pragma unroll 1
            for (int ps = 0; ps < NP; ++ps) {
              stage_rows(ps);
              __syncwarp();
              if (ps + 1 == NP) release();
              combine(ps, b0);
              __syncwarp();      // the tile is rewritten by the next pass
              if (ps + 1 < NP) fetch(ps + 1, b0);
            }
          }
          continue;
        }
        if (!mbar_wait(accf_bar(ab), ph, dead, p.status, p.spin_limit, 256)) { alive = false; break; }
        tc_fence_after();
#pragma unroll 1
        for (int sj = 0; sj < SLABS; ++sj) {
          // slab sj of the warps of one row quadrant lie side by side, so that the quadrant reads and
          // writes contiguous row segments of 32 * (EPI_WARPS / 4) columns at about the same time
          const int cb = sj * (C::EPI_WARPS / 4) + half;
          float acc[32];
          tmem_ld32(tmem_base + (uint32_t)(ab * ACCS * BN + cb * 32) + ((uint32_t)(quad * 32) << 16), acc);
          if (SPLIT) {
            float small[32];
            tmem_ld32(tmem_base + (uint32_t)(ab * ACCS * BN + BN + cb * 32) + ((uint32_t)(quad * 32) << 16), small);
#pragma unroll
            for (int e = 0; e < 32; ++e) acc[e] += small[e];
          }
          if (gi < g.M) {
            float4* cptr[8];
            float4 cur[8];
            bool ok[8];
            const bool to_part = p.splits > 1;
            const bool need_c = !first || (!to_part && g.epi != EPI_STORE && g.epi != EPI_C2_SUB);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const i64 col = n0 + cb * 32 + q * 4;
              ok[q] = col < g.N;
              cptr[q] = to_part ? reinterpret_cast<float4*>(partb + ((i64)it.ks * g.M + gi) * g.N + col)
                                : reinterpret_cast<float4*>(Cb + gi * g.ldc + col);
              cur[q] = make_float4(0.f, 0.f, 0.f, 0.f);
              if (ok[q] && need_c) cur[q] = *cptr[q];
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              if (!ok[q]) continue;
              const i64 col = n0 + cb * 32 + q * 4;
              float4 a4 = make_float4(acc[q * 4], acc[q * 4 + 1], acc[q * 4 + 2], acc[q * 4 + 3]);
              float4 c = cur[q];
              float sgn = 1.f, scale = 1.f;
              if (!to_part) {
                scale = alpha;
                if (g.epi != EPI_STORE) sgn = -1.f;
                if (first && (g.epi == EPI_ADD2_SUB || g.epi == EPI_C2_SUB)) {
                  if (g.c2_mode == ADD_F32 || g.epi == EPI_C2_SUB) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(C2b) + gi * g.ldc2 + col));
                    c.x += t.x; c.y += t.y; c.z += t.z; c.w += t.w;
                  } else {
                    const uint2 t = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(C2b) + gi * g.ldc2 + col));
                    const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&t.x);
                    const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&t.y);
                    c.x += __low2float(lo); c.y += __high2float(lo); c.z += __low2float(hi); c.w += __high2float(hi);
                  }
                }
              }
              const float f = sgn * scale;
              *cptr[q] = make_float4(fmaf(f, a4.x, c.x), fmaf(f, a4.y, c.y), fmaf(f, a4.z, c.z), fmaf(f, a4.w, c.w));
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (CG2 && cta_rank != 0) mbar_arrive_remote_relaxed(acce_bar(ab), 0u);
          else mbar_arrive(acce_bar(ab));
        }
      }
    }
  } else if (warp < C::MMA_WARP) {
    // ------------------------------------------------------------ producers
    const int ptid = threadIdx.x - NUM_EPI_WARPS * 32;
    if (NOCONV) {
      // nothing to convert: the TMA warp fills the operand tiles
    } else if (TMA) {
      // in-place conversion of the tiles the TMA warp loaded; the split is elementwise, so
      // each thread simply takes the 16-byte units ptid, ptid + 256, ... of the buffers
      const bool add = (g.a2_mode == ADD_F32);
      const bool add16 = (g.a2_mode == ADD_BF16);
      // bf16 addend: where the four bf16 values of each of this thread's A units sit in the
      // (unswizzled) staging tile; the unit index is un-swizzled back to (row, k)
      uint32_t g16off[C::A_CHUNKS];
#pragma unroll
      for (int l = 0; l < C::A_CHUNKS; ++l) {
        const uint32_t u = (uint32_t)ptid + l * NUM_PROD_THREADS;
        if (!A_MN) {
          const uint32_t row = u >> 3, minor = (u & 7u) ^ (row & 7u);
          g16off[l] = row * 64u + minor * 8u;
        } else {
          const uint32_t c = u >> 8, kk = (u >> 3) & 31u, qs = u & 7u;
          const uint32_t q = ((((qs >> 1) ^ (kk & 3u))) << 1) | (qs & 1u);
          g16off[l] = kk * 256u + (c * 32u + q * 4u) * 2u;
        }
      }
      // bf16 operands: byte offset of each unit's four bf16 values in the operand tile
      uint32_t aout[C::A_CHUNKS], bout[C::B_CHUNKS];
      if (C::BT) {
        auto out_off = [](uint32_t u, bool mn) -> uint32_t {
          if (!mn) {   // unit u = (row, swizzled 16-byte chunk) of a 128-byte fp32 row
            const uint32_t row = u >> 3, kc = (u & 7u) ^ (row & 7u);
            return row * 64u + ((((kc >> 1) ^ ((row >> 1) & 3u))) << 4) + (kc & 1u) * 8u;
          }
          // unit u = (32-row column chunk c, k row kk, swizzled unit qs): rows c*32 + q*4 .. +3 at k = kk
          const uint32_t c = u >> 8, kk = (u >> 3) & 31u, qs = u & 7u;
          const uint32_t q = ((((qs >> 1) ^ (kk & 3u))) << 1) | (qs & 1u);
          return (c >> 1) * (uint32_t)(BKE * 128) + kk * 128u + (((((c & 1u) << 2) | (q >> 1)) ^ (kk & 7u)) << 4) + (q & 1u) * 8u;
        };
#pragma unroll
        for (int l = 0; l < C::A_CHUNKS; ++l) aout[l] = out_off((uint32_t)ptid + l * NUM_PROD_THREADS, A_MN);
#pragma unroll
        for (int l = 0; l < C::B_CHUNKS; ++l) bout[l] = out_off((uint32_t)ptid + l * NUM_PROD_THREADS, B_MN);
      }
      int stage = 0;
      uint32_t phase = 0;
      bool alive = true;
      for (int item = worker; item < p.num_items && alive; item += workers) {
        const Item it = decode_item<BN, BKE, CG2>(p, item);
        if (skipped(it)) continue;
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait(raw_bar(stage), phase, dead, p.status, p.spin_limit)) { alive = false; break; }
          const uint32_t sg16 = g16_base + stage * C::G16_BYTES;
          const uint32_t sa = smem_base + stage * C::STAGE_BYTES + (uint32_t)ptid * 16u;
          const uint32_t sa_lo = sa + C::A_BYTES;
          const uint32_t sb = sa + 2 * C::A_BYTES;
          const uint32_t sb_lo = sb + C::B_BYTES;
          float4 xa[C::A_CHUNKS], ga[C::A_CHUNKS], xb[C::B_CHUNKS];
#pragma unroll
          for (int l = 0; l < C::A_CHUNKS; ++l) {
            xa[l] = lds128(sa + l * (NUM_PROD_THREADS * 16));
            if (add) ga[l] = lds128(sa_lo + l * (NUM_PROD_THREADS * 16));
            if (add16) {
              uint32_t w0, w1;
              asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(w0), "=r"(w1) : "r"(sg16 + g16off[l]) : "memory");
              const __nv_bfloat162 lo2 = *reinterpret_cast<const __nv_bfloat162*>(&w0);
              const __nv_bfloat162 hi2 = *reinterpret_cast<const __nv_bfloat162*>(&w1);
              ga[l] = make_float4(__low2float(lo2), __high2float(lo2), __low2float(hi2), __high2float(hi2));
            }
          }
#pragma unroll
          for (int l = 0; l < C::B_CHUNKS; ++l) xb[l] = lds128(sb + l * (NUM_PROD_THREADS * 16));
          if (C::BT) {
            const uint32_t a_out = smem_base + stage * C::STAGE_BYTES + 2 * C::A_BYTES + C::B_BYTES;
            const uint32_t b_out = a_out + C::A_BYTES / 2;
#pragma unroll
            for (int l = 0; l < C::A_CHUNKS; ++l) {
              float4 x = xa[l];
              if (add || add16) { x.x += ga[l].x; x.y += ga[l].y; x.z += ga[l].z; x.w += ga[l].w; }
              sts64_bf16x4(a_out + aout[l], x);
            }
#pragma unroll
            for (int l = 0; l < C::B_CHUNKS; ++l) sts64_bf16x4(b_out + bout[l], xb[l]);
          } else {
#pragma unroll
          for (int l = 0; l < C::A_CHUNKS; ++l) {
            float4 x = xa[l];
            if (add || add16) {
              x.x += ga[l].x; x.y += ga[l].y; x.z += ga[l].z; x.w += ga[l].w;
              sts128(sa + l * (NUM_PROD_THREADS * 16), x);
            }
            sts128(sa_lo + l * (NUM_PROD_THREADS * 16), make_float4(trunc_rem(x.x), trunc_rem(x.y), trunc_rem(x.z), trunc_rem(x.w)));
          }
#pragma unroll
          for (int l = 0; l < C::B_CHUNKS; ++l) {
            const float4 x = xb[l];
            sts128(sb_lo + l * (NUM_PROD_THREADS * 16), make_float4(trunc_rem(x.x), trunc_rem(x.y), trunc_rem(x.z), trunc_rem(x.w)));
          }
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            if (CG2 && cta_rank != 0) mbar_arrive_remote(full_bar(stage), 0u);
            else mbar_arrive(full_bar(stage));
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    } else {
    TileMap<BM, BKE, EPC, A_MN, C::A_CHUNKS, BF16> ma;
    TileMap<BN, BKE, EPC, B_MN, C::B_CHUNKS, BF16> mb;
    ma.init(ptid, g.a_si, g.a_sk, g.a2_si, g.a2_sk);
    mb.init(ptid, g.b_sn, g.b_sk, 0, 0);
    const int a2_elem = (g.a2_mode == ADD_BF16) ? 2 : 4;
    int stage = 0;
    uint32_t phase = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < p.num_items && alive; item += gridDim.x) {
      const Item it = decode_item<BN, BKE>(p, item);
      const i64 row0a = (i64)it.mi * BM, row0b = (i64)it.ni * BN;
      i64 k_end = g.K;
      if (g.klimit) k_end = min(g.K, (i64)(it.ni + 1) * BN);
      const float* a_row = g.A + row0a * g.a_si;
      const char* a2_row = reinterpret_cast<const char*>(g.A2) + row0a * g.a2_si * a2_elem;
      const float* b_row = g.B + row0b * g.b_sn;
      for (int kb = it.kb0; kb < it.kb1; ++kb) {
        const i64 k0 = (i64)kb * BKE;
        float va[C::A_CHUNKS][EPC], wa[C::A_CHUNKS][EPC];
        float vb[C::B_CHUNKS][EPC];
        ma.load(a_row + k0 * g.a_sk, a2_row + k0 * g.a2_sk * a2_elem, g.a2_mode, g.M - row0a, k_end - k0, va, wa);
        mb.load(b_row + k0 * g.b_sk, nullptr, ADD_NONE, g.N - row0b, k_end - k0, vb, vb);
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, dead, p.status, p.spin_limit)) { alive = false; break; }
        ma.add(g.a2_mode, va, wa);
        const uint32_t sa = smem_base + stage * C::STAGE_BYTES;
        const uint32_t sa_lo = sa + C::A_BYTES;
        const uint32_t sb = sa + (BF16 ? 1 : 2) * C::A_BYTES;
        const uint32_t sb_lo = sb + C::B_BYTES;
        ma.store(sa, sa_lo, va);
        mb.store(sb, sb_lo, vb);
        // every thread makes its own writes visible to the tensor core's (async) proxy, then
        // one lane per warp arrives: 8 arrivals per stage instead of 256 serialised ones
        fence_proxy_async();
        __syncwarp();
        const bool withheld = p.withhold_arrive != 0 && item == (int)blockIdx.x && kb == it.kb0;
        if (lane == 0 && !withheld) mbar_arrive(full_bar(stage));
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
    }
    }
  } else if (TMA && warp == C::MMA_WARP + 1) {
    // ------------------------------------------------------------ TMA issuer
    if (lane == 0) {
      const bool add = (g.a2_mode == ADD_F32);
      const bool add16 = (g.a2_mode == ADD_BF16);
      const uint32_t bytes = (uint32_t)(C::A_BYTES * (add ? 2 : 1) + C::B_BYTES + (add16 ? C::G16_BYTES : 0));
      int stage = 0;
      uint32_t phase = 0;
      bool alive = true;
      for (int item = worker; item < p.num_items && alive; item += workers) {
        const Item it = decode_item<BN, BKE, CG2>(p, item);
        if (skipped(it)) continue;
        // CTA pair: this CTA's 128 rows of A and its half of the B tile's columns
        const int row0a = (CG2 ? 2 * it.mi + (int)cta_rank : it.mi) * BM;
        const int row0b = it.ni * BN + (CG2 ? (int)cta_rank * BN_L : 0);
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, dead, p.status, p.spin_limit, 32)) { alive = false; break; }
          const int k0 = kb * BKE;
          const uint32_t sa = smem_base + stage * C::STAGE_BYTES;
          const uint32_t sa_lo = sa + C::A_BYTES;
          const uint32_t sb = sa + ((NOCONV && !X2) ? 1 : 2) * C::A_BYTES;
          const uint32_t bar = raw_bar(stage);
          // A pair without converter warps: both CTAs' tiles complete on the LEADER's barrier of the stage, which
          // its TMA thread arms for the bytes of both, and which its MMA thread waits on.  (A completion may reach
          // the barrier before it is armed: the phase still cannot end before the arming arrival.)  The peer's
          // loads for the stage's next use wait for the leader's commit, hence for the end of this phase.
          const uint32_t bar_pair = PAIRLOAD ? cluster_addr(bar, 0u) : bar;
          auto ld3 = [&](uint32_t dst, const CUtensorMap* map, int x, int y, int z) {
            if constexpr (PAIRLOAD) tma_load_3d_pair(dst, map, x, y, z, bar_pair);
            else tma_load_3d(dst, map, x, y, z, bar);
          };
          auto expect = [&](uint32_t nbytes) {
            if constexpr (PAIRLOAD) { if (cta_rank == 0) mbar_expect_tx(bar, 2u * nbytes); }
            else mbar_expect_tx(bar, nbytes);
          };
          if (X2) {   // hi and lo tiles of both operands: [rows][64 k] boxes, or [64 k][64 rows] boxes per 64-row chunk
            expect((uint32_t)(2 * (C::A_BYTES + C::B_BYTES)));
            const uint32_t sb_lo2 = sb + C::B_BYTES;
            if (!A_MN) {
              ld3(sa, &p.tmA, k0, row0a, it.b);
              ld3(sa_lo, &p.tmA2, k0, row0a, it.b);
            } else {
#pragma unroll
              for (int c = 0; c < BM / 64; ++c) {
                ld3(sa + c * (BKE * 128), &p.tmA, row0a + 64 * c, k0, it.b);
                ld3(sa_lo + c * (BKE * 128), &p.tmA2, row0a + 64 * c, k0, it.b);
              }
            }
            if (!B_MN) {
              ld3(sb, &p.tmB, k0, row0b, it.b);
              ld3(sb_lo2, &p.tmB2, k0, row0b, it.b);
            } else {
#pragma unroll
              for (int c = 0; c < BN_L / 64; ++c) {
                ld3(sb + c * (BKE * 128), &p.tmB, row0b + 64 * c, k0, it.b);
                ld3(sb_lo2 + c * (BKE * 128), &p.tmB2, row0b + 64 * c, k0, it.b);
              }
            }
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            continue;
          }
          if (ONE) {   // raw fp32 tiles, [rows][32 k] boxes
            expect((uint32_t)(C::A_BYTES + C::B_BYTES));
            ld3(sa, &p.tmA, k0, row0a, it.b);
            ld3(sb, &p.tmB, k0, row0b, it.b);
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            continue;
          }
          if (D16) {   // bf16 tiles: [rows][64 k] boxes, or [64 k][64 rows] boxes per 64-row chunk
            expect((uint32_t)(C::A_BYTES + C::B_BYTES));
            if (!A_MN) ld3(sa, &p.tmA, k0, row0a, it.b);
            else {
#pragma unroll
              for (int c = 0; c < BM / 64; ++c) ld3(sa + c * (BKE * 128), &p.tmA, row0a + 64 * c, k0, it.b);
            }
            if (!B_MN) ld3(sb, &p.tmB, k0, row0b, it.b);
            else {
#pragma unroll
              for (int c = 0; c < BN_L / 64; ++c) ld3(sb + c * (BKE * 128), &p.tmB, row0b + 64 * c, k0, it.b);
            }
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            continue;
          }
          mbar_expect_tx(bar, bytes);
          if (add16) {   // bf16 addend tile, unswizzled: [row][32 k] or [k][128 rows]
            if (!A_MN) tma_load_2d(g16_base + stage * C::G16_BYTES, &p.tmA2, k0, row0a, bar);
            else tma_load_2d(g16_base + stage * C::G16_BYTES, &p.tmA2, row0a, k0, bar);
          }
          if (!A_MN) {
            tma_load_3d(sa, &p.tmA, k0, row0a, it.b, bar);
            if (add) tma_load_3d(sa_lo, &p.tmA2, k0, row0a, it.b, bar);
          } else {
#pragma unroll
            for (int c = 0; c < BM / 32; ++c) {
              tma_load_3d(sa + c * (BKE * 128), &p.tmA, row0a + 32 * c, k0, it.b, bar);
              if (add) tma_load_3d(sa_lo + c * (BKE * 128), &p.tmA2, row0a + 32 * c, k0, it.b, bar);
            }
          }
          if (!B_MN) {
            tma_load_3d(sb, &p.tmB, k0, row0b, it.b, bar);
          } else {
#pragma unroll
            for (int c = 0; c < BN_L / 32; ++c) tma_load_3d(sb + c * (BKE * 128), &p.tmB, row0b + 32 * c, k0, it.b, bar);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ MMA issuer (CTA pair: the leader only)
    if (lane == 0 && (!CG2 || cta_rank == 0)) {
      const uint32_t idesc = make_idesc(BF16, A_MN, B_MN, BN, CG2 ? 2 * BM : BM, BF16 && p.g.f16 != 0);
      const uint32_t lbo = BKE * 128;
      constexpr uint32_t A_KSTEP = A_MN ? (BF16 ? 2048u : 1024u) : 32u;   // bytes per UMMA K step
      constexpr uint32_t B_KSTEP = B_MN ? (BF16 ? 2048u : 1024u) : 32u;
      int stage = 0;
      uint32_t phase = 0;
      int iter = 0;
      bool alive = true;
      for (int item = worker; item < p.num_items && alive; item += workers) {
        const Item it = decode_item<BN, BKE, CG2>(p, item);
        if (skipped(it)) continue;
        for (int kbc = it.kb0; kbc < it.kb1 && alive; kbc += p.kc, ++iter) {   // one accumulation chunk
        const int kbc1 = min(it.kb1, kbc + p.kc);
        const int ab = iter % NBUF;
        const uint32_t aph = (uint32_t)(iter / NBUF) & 1u;
        if (!mbar_wait<CG2>(acce_bar(ab), aph ^ 1u, dead, p.status, p.spin_limit, 64)) { alive = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(ab * ACCS * BN);
        const uint32_t d_small = d_tmem + (SPLIT ? BN : 0);
        uint32_t accumulate = 0;
        for (int kb = kbc; kb < kbc1; ++kb) {
          if (NOCONV) {   // this CTA's tiles (TMA) and, in a pair, the peer's (they complete on this barrier too)
            if (!mbar_wait<CG2>(raw_bar(stage), phase, dead, p.status, p.spin_limit)) { alive = false; break; }
          } else {
            if (!mbar_wait<CG2>(full_bar(stage), phase, dead, p.status, p.spin_limit)) { alive = false; break; }
          }
          tc_fence_after();
          const uint32_t st0 = smem_base + stage * C::STAGE_BYTES;
          // bf16 operands formed from TMA tiles sit behind the raw tiles of the stage
          const uint32_t sa = C::BT ? st0 + 2 * C::A_BYTES + C::B_BYTES : st0;
          const uint32_t sa_lo = sa + C::A_BYTES;
          const uint32_t sb = C::BT ? sa + C::A_BYTES / 2 : sa + (((BF16 && !X2) || ONE) ? 1 : 2) * C::A_BYTES;
          const uint32_t sb_lo = sb + C::B_BYTES;
#pragma unroll
          for (int ks = 0; ks < C::KSTEPS; ++ks) {
            const uint64_t a_hi = (C::BT && !A_MN) ? make_desc_k64(sa + ks * A_KSTEP) : make_desc<BF16>(sa + ks * A_KSTEP, A_MN, lbo);
            const uint64_t b_hi = (C::BT && !B_MN) ? make_desc_k64(sb + ks * B_KSTEP) : make_desc<BF16>(sb + ks * B_KSTEP, B_MN, lbo);
            if (X2) {
              const uint64_t a_lo = make_desc<BF16>(sa_lo + ks * A_KSTEP, A_MN, lbo);
              const uint64_t b_lo = make_desc<BF16>(sb_lo + ks * B_KSTEP, B_MN, lbo);
              // (split accumulators: the small terms in their own accumulator, one truncating add per K step on the main sum)
              if (CG2) {
                umma2_f16(d_small, a_hi, b_lo, idesc, accumulate);
                umma2_f16(d_small, a_lo, b_hi, idesc, 1u);
                umma2_f16(d_tmem, a_hi, b_hi, idesc, SPLIT ? accumulate : 1u);
              } else {
                umma<true>(d_small, a_hi, b_lo, idesc, accumulate);   // small terms first
                umma<true>(d_small, a_lo, b_hi, idesc, 1u);
                umma<true>(d_tmem, a_hi, b_hi, idesc, SPLIT ? accumulate : 1u);
              }
              accumulate = 1;
            } else if (BF16) {
              if (CG2) umma2_f16(d_tmem, a_hi, b_hi, idesc, accumulate);
              else umma<true>(d_tmem, a_hi, b_hi, idesc, accumulate);
              accumulate = 1;
            } else if (ONE) {
              umma<false>(d_tmem, a_hi, b_hi, idesc, accumulate);
              accumulate = 1;
            } else {
              const uint64_t a_lo = make_desc<BF16>(sa_lo + ks * A_KSTEP, A_MN, lbo);
              const uint64_t b_lo = make_desc<BF16>(sb_lo + ks * B_KSTEP, B_MN, lbo);
              if (CG2) {
                if (SPLIT) {
                  umma2_tf32(d_small, a_hi, b_lo, idesc, accumulate);
                  umma2_tf32(d_small, a_lo, b_hi, idesc, 1u);
                  umma2_tf32(d_small, a_lo, b_lo, idesc, 1u);
                  umma2_tf32(d_tmem, a_hi, b_hi, idesc, accumulate);
                } else {
                  umma2_tf32(d_tmem, a_hi, b_lo, idesc, accumulate);
                  umma2_tf32(d_tmem, a_lo, b_hi, idesc, 1u);
                  umma2_tf32(d_tmem, a_hi, b_hi, idesc, 1u);
                }
              } else if (SPLIT) {
                umma<false>(d_small, a_hi, b_lo, idesc, accumulate);
                umma<false>(d_small, a_lo, b_hi, idesc, 1u);
                // truncation remainders all carry the sign of their operand: lo * lo is not noise
                if (TMA) umma<false>(d_small, a_lo, b_lo, idesc, 1u);
                umma<false>(d_tmem, a_hi, b_hi, idesc, accumulate);
              } else {
                umma<false>(d_tmem, a_hi, b_lo, idesc, accumulate);   // small terms first
                umma<false>(d_tmem, a_lo, b_hi, idesc, 1u);
                umma<false>(d_tmem, a_hi, b_hi, idesc, 1u);
              }
              accumulate = 1;
            }
          }
          if (CG2) umma2_commit(empty_bar(stage), (uint16_t)3);   // both CTAs may refill the stage
          else umma_commit(empty_bar(stage));   // the stage may be refilled once these MMAs are done
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!alive) break;
        if (CG2) umma2_commit(accf_bar(ab), (uint16_t)3);   // each CTA's epilogue reads its own half
        else umma_commit(accf_bar(ab));         // this chunk's accumulator is complete
        }
      }
      // drain: every issued MMA must have finished before TMEM is released
      if (CG2) umma2_commit(drain_bar, (uint16_t)1);
      else umma_commit(drain_bar);
      mbar_wait(drain_bar, 0u, dead, p.status, p.spin_limit, 64);
    }
    __syncwarp();
  }

  tc_fence_before();
  __syncthreads();
  // CTA pair: neither CTA may leave (or free its accumulators) while the other still arrives on its barriers
  // or the leader's MMAs still read its shared memory
  if (CG2) cluster_sync_all();
  if (warp == C::MMA_WARP) {
    tc_fence_after();
    if (CG2) tmem_dealloc2(tmem_base, C::TMEM_COLS);
    else tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

template <int BN, bool A_MN, bool B_MN, bool BF16, bool SPLIT, bool TMA, bool D16 = false, bool CE = false, bool ONE = false,
          bool CG2 = false, bool X2 = false>
inline cudaError_t set_smem_attr() {
  return cudaFuncSetAttribute(k_gemm_umma<BN, A_MN, B_MN, BF16, SPLIT, TMA, D16, CE, ONE, CG2, X2>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Cfg<BN, BF16, SPLIT, TMA, D16, CE, ONE, CG2, X2>::SMEM_BYTES);
}

// bf16 operand pairs
template <int BN, bool A_MN, bool B_MN>
inline void launch_x2_one(const Params& p, int grid, cudaStream_t st) {
  constexpr int smem = Cfg<BN, true, false, true, true, true, false, false, true>::SMEM_BYTES;
  constexpr int threads = Cfg<BN, true, false, true, true, true, false, false, true>::THREADS;
  k_gemm_umma<BN, A_MN, B_MN, true, false, true, true, true, false, false, true><<<grid, threads, smem, st>>>(p);
}
template <int BN>
inline void launch_x2(const Params& p, bool a_mn, bool b_mn, int grid, cudaStream_t st) {
  if (!a_mn && !b_mn) launch_x2_one<BN, false, false>(p, grid, st);
  else if (!a_mn && b_mn) launch_x2_one<BN, false, true>(p, grid, st);
  else if (a_mn && b_mn) launch_x2_one<BN, true, true>(p, grid, st);
  else launch_x2_one<BN, true, false>(p, grid, st);
}
template <int BN, bool A_MN, bool B_MN>
inline cudaError_t set_x2_attr() {
  return set_smem_attr<BN, A_MN, B_MN, true, false, true, true, true, false, false, true>();
}

// operand pairs with split accumulators: B row-index contiguous (Gram matrices: A too; P = (M + G) Q: A k-contiguous)
template <int BN, bool A_MN>
inline void launch_x2s(const Params& p, int grid, cudaStream_t st) {
  using CF = Cfg<BN, true, true, true, true, true, false, false, true>;
  k_gemm_umma<BN, A_MN, true, true, true, true, true, true, false, false, true><<<grid, CF::THREADS, CF::SMEM_BYTES, st>>>(p);
}
template <bool A_MN>
inline cudaError_t launch_x2s_pair(const Params& p, int grid, cudaStream_t st) {
  using CF = Cfg<256, true, true, true, true, true, false, true, true>;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(CF::THREADS); cfg.dynamicSmemBytes = CF::SMEM_BYTES; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_gemm_umma<256, A_MN, true, true, true, true, true, true, false, true, true>, p);
}

// bf16 operand pairs on CTA pairs
template <bool A_MN, bool B_MN>
inline cudaError_t launch_x2_pair_one(const Params& p, int grid, cudaStream_t st) {
  using CF = Cfg<256, true, false, true, true, true, false, true, true>;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(CF::THREADS); cfg.dynamicSmemBytes = CF::SMEM_BYTES; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_gemm_umma<256, A_MN, B_MN, true, false, true, true, true, false, true, true>, p);
}
inline cudaError_t launch_x2_pair(const Params& p, bool a_mn, bool b_mn, int grid, cudaStream_t st) {
  if (!a_mn && !b_mn) return launch_x2_pair_one<false, false>(p, grid, st);
  if (!a_mn && b_mn) return launch_x2_pair_one<false, true>(p, grid, st);
  if (a_mn && b_mn) return launch_x2_pair_one<true, true>(p, grid, st);
  return launch_x2_pair_one<true, false>(p, grid, st);
}
template <bool A_MN, bool B_MN>
inline cudaError_t set_x2_pair_attr() {
  return set_smem_attr<256, A_MN, B_MN, true, false, true, true, true, false, true, true>();
}

// 16-bit arrays (one array per operand) on CTA pairs
template <bool A_MN, bool B_MN>
inline cudaError_t launch_d16_pair_one(const Params& p, int grid, cudaStream_t st) {
  using CF = Cfg<256, true, false, true, true, true, false, true, false>;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(CF::THREADS); cfg.dynamicSmemBytes = CF::SMEM_BYTES; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_gemm_umma<256, A_MN, B_MN, true, false, true, true, true, false, true, false>, p);
}
inline cudaError_t launch_d16_pair(const Params& p, bool a_mn, bool b_mn, int grid, cudaStream_t st) {
  if (!a_mn && !b_mn) return launch_d16_pair_one<false, false>(p, grid, st);
  if (!a_mn && b_mn) return launch_d16_pair_one<false, true>(p, grid, st);
  if (a_mn && b_mn) return launch_d16_pair_one<true, true>(p, grid, st);
  return launch_d16_pair_one<true, false>(p, grid, st);
}
template <bool A_MN, bool B_MN>
inline cudaError_t set_d16_pair_attr() {
  return set_smem_attr<256, A_MN, B_MN, true, false, true, true, true, false, true, false>();
}

// CTA pairs: clusters of two CTAs, 256 x 256 tiles (fp32 mode, TMA, coalesced epilogue)
template <bool A_MN, bool B_MN, bool SPLIT>
inline cudaError_t launch_pair_one(const Params& p, int grid, cudaStream_t st) {
  constexpr int smem = Cfg<256, false, SPLIT, true, false, true, false, true>::SMEM_BYTES;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(NUM_THREADS_TMA); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_gemm_umma<256, A_MN, B_MN, false, SPLIT, true, false, true, false, true>, p);
}
template <bool SPLIT>
inline cudaError_t launch_pair(const Params& p, bool a_mn, bool b_mn, int grid, cudaStream_t st) {
  if (!a_mn && !b_mn) return launch_pair_one<false, false, SPLIT>(p, grid, st);
  if (!a_mn && b_mn) return launch_pair_one<false, true, SPLIT>(p, grid, st);
  if (a_mn && b_mn) return launch_pair_one<true, true, SPLIT>(p, grid, st);
  return launch_pair_one<true, false, SPLIT>(p, grid, st);
}
template <bool A_MN, bool B_MN>
inline cudaError_t set_pair_attr() {
  cudaError_t e = set_smem_attr<256, A_MN, B_MN, false, false, true, false, true, false, true>();
  if (e == cudaSuccess) e = set_smem_attr<256, A_MN, B_MN, false, true, true, false, true, false, true>();
  return e;
}
// How many CTA pairs can be resident at once (per device, asked once).
inline int pair_clusters(int sm_count) {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return sm_count / 2; }
  if (dev >= 0 && dev < 64 && cached[dev] > 0) return cached[dev];
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(sm_count / 2 * 2)); cfg.blockDim = dim3(NUM_THREADS_TMA);
  cfg.dynamicSmemBytes = Cfg<256, false, false, true, false, true, false, true>::SMEM_BYTES;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, k_gemm_umma<256, false, false, false, false, true, false, true, false, true>, &cfg) != cudaSuccess ||
      n < 1) {
    cudaGetLastError();
    n = 0;
  }
  if (n > sm_count / 2) n = sm_count / 2;
  if (dev >= 0 && dev < 64) cached[dev] = n > 0 ? n : -1;
  return n;
}

// single-pass TF32 (k-contiguous operands only)
template <int BN>
inline void launch_one(const Params& p, int grid, cudaStream_t st) {
  constexpr int smem = Cfg<BN, false, false, true, false, true, true>::SMEM_BYTES;
  k_gemm_umma<BN, false, false, false, false, true, false, true, true><<<grid, NUM_THREADS_TMA, smem, st>>>(p);
}

template <int BN, bool BF16, bool SPLIT, bool TMA, bool D16 = false, bool CE = false>
inline void launch_variant(const Params& p, bool a_mn, bool b_mn, int grid, cudaStream_t st) {
  constexpr int smem = Cfg<BN, BF16, SPLIT, TMA, D16, CE>::SMEM_BYTES;
  constexpr int threads = TMA ? NUM_THREADS_TMA : NUM_THREADS;
  if (!a_mn && !b_mn) k_gemm_umma<BN, false, false, BF16, SPLIT, TMA, D16, CE><<<grid, threads, smem, st>>>(p);
  else if (!a_mn && b_mn) k_gemm_umma<BN, false, true, BF16, SPLIT, TMA, D16, CE><<<grid, threads, smem, st>>>(p);
  else if (a_mn && b_mn) k_gemm_umma<BN, true, true, BF16, SPLIT, TMA, D16, CE><<<grid, threads, smem, st>>>(p);
  else k_gemm_umma<BN, true, false, BF16, SPLIT, TMA, D16, CE><<<grid, threads, smem, st>>>(p);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, resolved once through the runtime (no link against libcuda).
inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
    else
      cudaGetLastError();
  }
  return fn;
}

// Tensor map of an fp32 operand tile source.  `rows` x `K` logical operand (row = M/N index).
// mn_major = false: memory is [rows][K] with row stride `ld`; box = 32 k x box_rows rows,
//   128-byte swizzle.  mn_major = true: memory is [K][rows] with k stride `ld`; box = 32
//   rows x 32 k, 128-byte swizzle with 32-byte atoms (the layout the TF32 MMA reads for a
//   row-contiguous operand).
// Tensor map of the bf16 addend of A: unswizzled tiles, [128 rows][32 k] (k contiguous) or
// [32 k][128 rows] (row index contiguous).
inline bool make_addend16_map(CUtensorMap* map, const void* ptr, i64 rows, i64 K, i64 ld, bool mn_major) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  cuuint64_t gdim[2], gstride[1];
  cuuint32_t box[2], estr[2] = {1, 1};
  if (!mn_major) { gdim[0] = (cuuint64_t)K; gdim[1] = (cuuint64_t)rows; box[0] = 32; box[1] = BM; }
  else { gdim[0] = (cuuint64_t)rows; gdim[1] = (cuuint64_t)K; box[0] = BM; box[1] = 32; }
  gstride[0] = (cuuint64_t)ld * 2;
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Tensor map of a bf16 operand: box = 64 k x box_rows rows (k contiguous) or 64 rows x 64 k
// (row index contiguous), 128-byte swizzle: exactly the tile the bf16 MMA reads.
// (3-D like the fp32 operand maps; `bstride_bytes` between the matrices of a batched launch)
inline bool make_operand16_map(CUtensorMap* map, const void* ptr, i64 rows, i64 K, i64 ld, bool mn_major, int box_rows,
                               i64 nbatch = 1, i64 bstride_bytes = 0) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  cuuint64_t gdim[3], gstride[2];
  cuuint32_t box[3], estr[3] = {1, 1, 1};
  if (!mn_major) { gdim[0] = (cuuint64_t)K; gdim[1] = (cuuint64_t)rows; box[0] = 64; box[1] = (cuuint32_t)box_rows; }
  else { gdim[0] = (cuuint64_t)rows; gdim[1] = (cuuint64_t)K; box[0] = 64; box[1] = 64; }
  gdim[2] = (cuuint64_t)(nbatch > 1 ? nbatch : 1);
  box[2] = 1;
  gstride[0] = (cuuint64_t)ld * 2;
  gstride[1] = (nbatch > 1) ? (cuuint64_t)bstride_bytes : gstride[0] * gdim[1];
  if (gstride[1] % 16 != 0) return false;
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), gdim, gstride, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// The maps of fp32 operands are 3-D: the third coordinate is the matrix of a batched launch (`nbatch` matrices,
// `bstride` elements apart; extent 1 otherwise).
inline bool make_operand_map(CUtensorMap* map, const void* ptr, i64 rows, i64 K, i64 ld, bool mn_major, int box_rows,
                             i64 nbatch = 1, i64 bstride = 0) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  cuuint64_t gdim[3], gstride[2];
  cuuint32_t box[3], estr[3] = {1, 1, 1};
  if (!mn_major) {
    gdim[0] = (cuuint64_t)K; gdim[1] = (cuuint64_t)rows;
    box[0] = 32; box[1] = (cuuint32_t)box_rows;
  } else {
    gdim[0] = (cuuint64_t)rows; gdim[1] = (cuuint64_t)K;
    box[0] = 32; box[1] = 32;
  }
  gdim[2] = (cuuint64_t)(nbatch > 1 ? nbatch : 1);
  box[2] = 1;
  gstride[0] = (cuuint64_t)ld * sizeof(float);
  gstride[1] = (nbatch > 1) ? (cuuint64_t)bstride * sizeof(float) : gstride[0] * gdim[1];
  if (gstride[1] % 16 != 0) return false;
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(ptr), gdim, gstride, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE,
                        mn_major ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace umma

// One-time set-up of the tensor-core kernels: opt in to their dynamic shared memory.
inline int umma_configure() {
  using namespace umma;
  // function attributes belong to a device's context: once per device of this process
  static bool done_on[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return DION_ERR_CUDA; }
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && done_on[dev]) return DION_OK;
  cudaError_t e = cudaSuccess;
#define DION_SET(BN, A, B, F)                                              \
  if (e == cudaSuccess) e = set_smem_attr<BN, A, B, F, false, false>();    \
  if (e == cudaSuccess && !F) e = set_smem_attr<BN, A, B, false, true, false>();  \
  if (e == cudaSuccess && !F) e = set_smem_attr<BN, A, B, false, false, true>();  \
  if (e == cudaSuccess && !F) e = set_smem_attr<BN, A, B, false, true, true>();  \
  if (e == cudaSuccess && F) e = set_smem_attr<BN, A, B, true, false, true>();    \
  if (e == cudaSuccess && F) e = set_smem_attr<BN, A, B, true, false, true, true, true>();  \
  if (e == cudaSuccess && !F) e = set_smem_attr<BN, A, B, false, false, true, false, true>();  \
  if (e == cudaSuccess && !F) e = set_smem_attr<BN, A, B, false, true, true, false, true>();
  DION_SET(128, false, false, false) DION_SET(128, false, true, false) DION_SET(128, true, true, false) DION_SET(128, true, false, false)
  DION_SET(256, false, false, false) DION_SET(256, false, true, false) DION_SET(256, true, true, false) DION_SET(256, true, false, false)
  DION_SET(128, false, false, true) DION_SET(128, false, true, true) DION_SET(128, true, true, true) DION_SET(128, true, false, true)
  DION_SET(256, false, false, true) DION_SET(256, false, true, true) DION_SET(256, true, true, true) DION_SET(256, true, false, true)
#undef DION_SET
  if (e == cudaSuccess) e = set_smem_attr<128, false, false, false, false, true, false, true, true>();
  if (e == cudaSuccess) e = set_smem_attr<256, false, false, false, false, true, false, true, true>();
  if (e == cudaSuccess) e = set_x2_attr<128, false, false>();
  if (e == cudaSuccess) e = set_x2_attr<128, false, true>();
  if (e == cudaSuccess) e = set_x2_attr<128, true, true>();
  if (e == cudaSuccess) e = set_x2_attr<128, true, false>();
  if (e == cudaSuccess) e = set_x2_attr<256, false, false>();
  if (e == cudaSuccess) e = set_x2_attr<256, false, true>();
  if (e == cudaSuccess) e = set_x2_attr<256, true, true>();
  if (e == cudaSuccess) e = set_x2_attr<256, true, false>();
  if (e == cudaSuccess) e = set_smem_attr<128, true, true, true, true, true, true, true, false, false, true>();
  if (e == cudaSuccess) e = set_smem_attr<256, true, true, true, true, true, true, true, false, false, true>();
  if (e == cudaSuccess) e = set_smem_attr<256, true, true, true, true, true, true, true, false, true, true>();
  if (e == cudaSuccess) e = set_smem_attr<128, false, true, true, true, true, true, true, false, false, true>();
  if (e == cudaSuccess) e = set_smem_attr<256, false, true, true, true, true, true, true, false, false, true>();
  if (e == cudaSuccess) e = set_smem_attr<256, false, true, true, true, true, true, true, false, true, true>();
  if (e == cudaSuccess) e = set_x2_pair_attr<false, false>();
  if (e == cudaSuccess) e = set_x2_pair_attr<false, true>();
  if (e == cudaSuccess) e = set_x2_pair_attr<true, true>();
  if (e == cudaSuccess) e = set_x2_pair_attr<true, false>();
  if (e == cudaSuccess) e = set_d16_pair_attr<false, false>();
  if (e == cudaSuccess) e = set_d16_pair_attr<false, true>();
  if (e == cudaSuccess) e = set_d16_pair_attr<true, true>();
  if (e == cudaSuccess) e = set_d16_pair_attr<true, false>();
  if (e == cudaSuccess) e = set_pair_attr<false, false>();
  if (e == cudaSuccess) e = set_pair_attr<false, true>();
  if (e == cudaSuccess) e = set_pair_attr<true, true>();
  if (e == cudaSuccess) e = set_pair_attr<true, false>();
  if (e != cudaSuccess) { cudaGetLastError(); return DION_ERR_CUDA; }
  if (tracked) done_on[dev] = true;
  return DION_OK;
}

// Launches the product on the tensor cores if it qualifies.  Returns the number of
// kernels launched (1, or 2 with a split-K reduction), 0 if this engine does not take
// the product, or a negative DION_ERR_* code.
// `variant` (test hook, 0 in the product): UMMA_VARIANT_* bits.
enum : int {
  UMMA_VARIANT_REGISTER_LOADS = 1,   // operands through registers instead of TMA
  UMMA_VARIANT_WITHHOLD = 2,         // with register loads: withhold one producer arrival, 1 ms wait budget
  UMMA_VARIANT_NO_PAIRS = 4          // single-CTA tiles where the product would take CTA pairs
};
constexpr i64 PAIR_MIN_ROWS = 512;   // smallest output height given to CTA pairs
constexpr i64 PAIR_MIN_TRI = 2048;   // smallest lower-triangular output given to CTA pairs
inline int umma_try_launch(const GemmArgs& g_in, int precision, int sm_count, float* part, i64 part_floats,
                           int* status, cudaStream_t st, int variant = 0) {
  using namespace umma;
  GemmArgs g = g_in;
  const bool d16 = g.ab16 != 0;      // bf16 operands in memory
  const bool bf16 = d16 || (precision == DION_PREC_BF16_OPERANDS);
  const int epc = bf16 ? 8 : 4;
  const int sm = d16 ? 8 : 4;        // stride granularity: 16 bytes
  if (g.batch != 1) return 0;
  // one launch over the matrices of a chain (same shape; operands, output and split-K scratch g.bs2 4-byte words
  // apart): operands through 3-D tensor maps only.  Tiles and K splits are chosen exactly as for one matrix,
  // so every element is computed by the same sequence of operations as in a launch of its own.
  const int nbat = g.batch2 > 1 ? g.batch2 : 1;
  if (nbat > 1 && (g.a2_mode == ADD_BF16 || (variant & UMMA_VARIANT_REGISTER_LOADS) || (g.bs2 % 4))) return 0;
  if ((g.c_tab != nullptr || g.c2_tab != nullptr) && (nbat < 2 || nbat > GEMM_TAB_MAX)) return 0;
  if (g.c_tab != nullptr && g.epi == EPI_STORE) return 0;   // (a plain store may split K: its reduction wants one stride)
  if (g.M < 128 || g.N < 64 || g.K < 64) return 0;
  if ((g.M % epc) || (g.N % epc) || (g.K % epc)) return 0;
  if (d16 && g.a2_mode != ADD_NONE) return 0;
  auto aligned = [](const void* p, size_t a) { return ((uintptr_t)p % a) == 0; };
  bool a_mn, b_mn;
  if (g.a_sk == 1 && g.a_si % sm == 0) a_mn = false;
  else if (g.a_si == 1 && g.a_sk % sm == 0) a_mn = true;
  else return 0;
  if (g.b_sk == 1 && g.b_sn % sm == 0) b_mn = false;
  else if (g.b_sn == 1 && g.b_sk % sm == 0) b_mn = true;
  else return 0;
  if (!aligned(g.A, 16) || !aligned(g.B, 16) || !aligned(g.C, 16) || (g.ldc % 4)) return 0;
  if (g.c_tab != nullptr)
    for (int b = 0; b < nbat; ++b)
      if (!aligned(g.c_tab[b], 16)) return 0;
  if (g.a2_mode != ADD_NONE) {
    if (a_mn ? (g.a2_si != 1 || g.a2_sk % 4) : (g.a2_sk != 1 || g.a2_si % 4)) return 0;
    if (!aligned(g.A2, g.a2_mode == ADD_BF16 ? 8 : 16)) return 0;
  }
  if (g.epi == EPI_ADD2_SUB || g.epi == EPI_C2_SUB) {
    const size_t al2 = (g.epi == EPI_ADD2_SUB && g.c2_mode == ADD_BF16) ? 8 : 16;
    if ((g.ldc2 % 4) || !aligned(g.C2, al2)) return 0;
    if (g.c2_tab != nullptr)
      for (int b = 0; b < nbat; ++b)
        if (!aligned(g.c2_tab[b], al2)) return 0;
  }
  if (g.tri == TRI_LOWER && g.M != g.N) return 0;

  // lower-triangular output: 128 x 256 tiles (more flops per operand byte; the tiles on the diagonal
  // compute up to 128 columns too many) once the matrix has enough tile rows for that to pay
  const bool tri_wide = g.tri == TRI_LOWER && g.epi == EPI_STORE && g.N >= TRI_WIDE_MIN;
  // CTA pairs (cta_group::2, 256 x 256 tiles): the fp32 (3xTF32) products that the TMA variant with the
  // coalesced epilogue takes, once the output is tall enough to give every pair work
  const int nclusters = pair_clusters(sm_count);
  // ... and the products on bf16 operand pairs (two thirds of the operand traffic per CTA, three stages instead of two)
  const bool x2 = d16 && g.A16lo != nullptr && g.B16lo != nullptr;   // bf16 operand pairs
  // ... and those on single 16-bit arrays (the operand tiles a CTA reads from L2 are what bounds them on single CTAs).
  // (Not the single-pass TF32 product, which only ragged shapes still take.)
  bool cg2 = ((!bf16 && !g.tf32x1 && g.a2_mode != ADD_BF16) || d16) &&
             !(variant & (UMMA_VARIANT_REGISTER_LOADS | UMMA_VARIANT_NO_PAIRS)) && nclusters > 0 &&
             g.N >= 256 && g.M >= PAIR_MIN_ROWS && (g.tri != TRI_LOWER || g.N >= PAIR_MIN_TRI);
  const int BN = ((g.tri == TRI_LOWER && !tri_wide && !cg2) || g.N < 256) ? 128 : 256;
  Params p;
  p.g = g;
  if (g.c_tab != nullptr) for (int b = 0; b < nbat; ++b) p.ctab[b] = g.c_tab[b];
  if (g.c2_tab != nullptr) for (int b = 0; b < nbat; ++b) p.c2tab[b] = g.c2_tab[b];
  // TMA variant: fp32 operands in memory (both precision modes), dimensions the tensor maps can describe
  bool tma = (d16 || !(variant & UMMA_VARIANT_REGISTER_LOADS)) && g.M < (1ll << 31) && g.N < (1ll << 31) && g.K < (1ll << 31);
  if (x2 && (!aligned(g.A16lo, 16) || !aligned(g.B16lo, 16))) return 0;
  if (d16) {
    const i64 lda = a_mn ? g.a_sk : g.a_si, ldb = b_mn ? g.b_sk : g.b_sn;
    const i64 bsb = g.bs2 * 4;   // the batch stride counts 4-byte words for every operand type
    if (!tma || !make_operand16_map(&p.tmA, g.A, g.M, g.K, lda, a_mn, BM, nbat, bsb) ||
        !make_operand16_map(&p.tmB, g.B, g.N, g.K, ldb, b_mn, cg2 ? BN / 2 : BN, nbat, bsb))
      return 0;
    if (x2 && (!make_operand16_map(&p.tmA2, g.A16lo, g.M, g.K, lda, a_mn, BM, nbat, bsb) ||
               !make_operand16_map(&p.tmB2, g.B16lo, g.N, g.K, ldb, b_mn, cg2 ? BN / 2 : BN, nbat, bsb)))
      return 0;
  } else
  if (tma && g.a2_mode == ADD_BF16) {   // the bf16 addend needs 16-byte aligned rows for its tensor map
    const i64 ld2 = a_mn ? g.a2_sk : g.a2_si;
    tma = (ld2 % 8 == 0) && (((uintptr_t)g.A2 % 16) == 0) &&
          make_addend16_map(&p.tmA2, g.A2, g.M, g.K, ld2, a_mn);
  }
  if (tma && !d16) {
    const i64 lda = a_mn ? g.a_sk : g.a_si, ldb = b_mn ? g.b_sk : g.b_sn;
    tma = make_operand_map(&p.tmA, g.A, g.M, g.K, lda, a_mn, BM, nbat, g.bs2) &&
          make_operand_map(&p.tmB, g.B, g.N, g.K, ldb, b_mn, cg2 ? BN / 2 : BN, nbat, g.bs2);
    if (tma && g.a2_mode == ADD_F32)
      tma = make_operand_map(&p.tmA2, g.A2, g.M, g.K, a_mn ? g.a2_sk : g.a2_si, a_mn, BM, nbat, g.bs2);
  }
  if (nbat > 1 && !tma) return 0;
  const int bke = (bf16 && (!tma || d16)) ? 64 : 32;
  if (cg2 && !tma) {   // no tensor maps: the register path knows no pairs; redo the tile choice without them
    GemmArgs g2 = g_in;
    return umma_try_launch(g2, precision, sm_count, part, part_floats, status, st, variant | UMMA_VARIANT_NO_PAIRS);
  }
  const int tile_m = cg2 ? 2 * BM : BM;
  p.nM = (int)((g.M + tile_m - 1) / tile_m);
  p.nN = (int)((g.N + BN - 1) / BN);
  p.nkb = (int)((g.K + bke - 1) / bke);
  const i64 tiles = (g.tri != TRI_LOWER) ? (i64)p.nM * p.nN
                    : (BN == 256 && !cg2)  ? ((i64)p.nM + 1) * (p.nM + 1) / 4
                                           : (i64)p.nM * (p.nM + 1) / 2;
  const int workers_max = cg2 ? nclusters : sm_count;   // CTAs, or CTA pairs, that can run at once
  // Tile order.  Row by row, a wave of tiles reads every column block of B; when B (N x K) is larger than what L2
  // keeps, every wave fetches it from DRAM again (ncu, X update at 16384^2, r = 4096: 16.8 GB read for 1.3 GB of
  // operands and output).  Then the output is walked in column panels whose B blocks (~32 MB) stay in L2.
  p.raster_gw = 0;
  if (g.tri != TRI_LOWER) {
    // DRAM bytes of the operands under either order (A block = one tile row of A, B block = one tile column of B;
    // L2 keeps ~60 MB of a re-read operand, a panel is held to 40 MB): row by row A is read once and B once per
    // wave unless it fits; in panels of gw columns B is read once and A once per panel
    const double esz = d16 ? (x2 ? 4.0 : 2.0) : 4.0;             // bytes per operand element as read by this variant
    const double ablock = (double)tile_m * (double)g.K * esz, bblock = (double)BN * (double)g.K * esz;
    const double nM = p.nM, nN = p.nN, W = workers_max;
    const double waves = nM * nN / W;
    const double by_rows = nM * ablock + ((nN * bblock > 60e6) ? waves * (nN < W ? nN : W) * bblock : nN * bblock);
    double best = 0.8 * by_rows;      // panels only for a clear gain
    for (int gw = 2; gw < p.nN && gw * bblock <= 40e6; ++gw) {
      const double cost = nM * ablock * (double)((p.nN + gw - 1) / gw) + nN * bblock;
      if (cost < best) { best = cost; p.raster_gw = gw; }
    }
  }
  int splits = 1;
  if (g.epi == EPI_STORE && !g.klimit && part != nullptr && tiles < workers_max) {
    i64 want = workers_max / tiles;
    const i64 kmax = p.nkb / 4;                       // at least four K blocks per split
    if (want > kmax) want = kmax;
    if (want > 32) want = 32;
    while (want > 1 && want * g.M * g.N > part_floats) --want;
    if (want > 1) splits = (int)want;
  }
  p.kb_per_split = (p.nkb + splits - 1) / splits;
  splits = (p.nkb + p.kb_per_split - 1) / p.kb_per_split;   // no empty split
  p.splits = splits;
  p.g.part = part;
  if (tiles * splits * nbat > 0x7fffffff) return 0;
  p.items_per_matrix = (int)(tiles * splits);
  p.num_items = p.items_per_matrix * nbat;
  p.status = status;
  const bool withhold = (variant & UMMA_VARIANT_WITHHOLD) && !tma;
  p.spin_limit = withhold ? 2000000LL : SPIN_LIMIT_CYCLES;
  p.withhold_arrive = withhold ? 1 : 0;
  // 32 K blocks per accumulation chain: 1024 k (8e-6 relative error in fp32 mode, 1.4e-6 with
  // split accumulators); 2048 k for bf16 operands loaded through registers
  p.kc = (x2 && (g.precise || g.f16)) ? 16 : 32;   // (K blocks of 64 there: the same 1024 k per chain as the fp32 products)
  const int grid = cg2 ? 2 * (p.num_items < nclusters ? p.num_items : nclusters)
                       : (p.num_items < sm_count ? p.num_items : sm_count);
  const bool one = g.tf32x1 && !bf16 && tma && !a_mn && !b_mn && g.a2_mode == ADD_NONE && !g.precise && splits == 1;
  if (x2 && g.precise) {   // (built with split accumulators for B row-index contiguous: Gram matrices and P)
    if (!b_mn) return 0;
    if (cg2) {
      const cudaError_t e = a_mn ? launch_x2s_pair<true>(p, grid, st) : launch_x2s_pair<false>(p, grid, st);
      if (e != cudaSuccess) { cudaGetLastError(); return DION_ERR_CUDA; }
    } else if (BN == 256) {
      if (a_mn) launch_x2s<256, true>(p, grid, st); else launch_x2s<256, false>(p, grid, st);
    } else {
      if (a_mn) launch_x2s<128, true>(p, grid, st); else launch_x2s<128, false>(p, grid, st);
    }
  } else if (cg2 && x2) {
    if (launch_x2_pair(p, a_mn, b_mn, grid, st) != cudaSuccess) { cudaGetLastError(); return DION_ERR_CUDA; }
  } else if (cg2 && d16) {
    if (launch_d16_pair(p, a_mn, b_mn, grid, st) != cudaSuccess) { cudaGetLastError(); return DION_ERR_CUDA; }
  } else if (cg2) {
    const cudaError_t e = g.precise ? launch_pair<true>(p, a_mn, b_mn, grid, st) : launch_pair<false>(p, a_mn, b_mn, grid, st);
    if (e != cudaSuccess) { cudaGetLastError(); return DION_ERR_CUDA; }
  } else if (one) {
    if (BN == 256) launch_one<256>(p, grid, st);
    else launch_one<128>(p, grid, st);
  } else if (x2) {
    if (BN == 256) launch_x2<256>(p, a_mn, b_mn, grid, st);
    else launch_x2<128>(p, a_mn, b_mn, grid, st);
  } else if (d16) {   // bf16 arrays: always with the coalesced epilogue
    if (BN == 256) launch_variant<256, true, false, true, true, true>(p, a_mn, b_mn, grid, st);
    else launch_variant<128, true, false, true, true, true>(p, a_mn, b_mn, grid, st);
  } else if (bf16 && tma) {
    if (BN == 256) launch_variant<256, true, false, true>(p, a_mn, b_mn, grid, st);
    else launch_variant<128, true, false, true>(p, a_mn, b_mn, grid, st);
  } else if (bf16) {
    if (BN == 256) launch_variant<256, true, false, false>(p, a_mn, b_mn, grid, st);
    else launch_variant<128, true, false, false>(p, a_mn, b_mn, grid, st);
  } else if (tma && g.a2_mode != ADD_BF16 && (!g.precise || BN == 256 || g.epi != EPI_STORE)) {   // coalesced epilogue in place of the bf16 addend staging
    if (g.precise) {
      if (BN == 256) launch_variant<256, false, true, true, false, true>(p, a_mn, b_mn, grid, st);
      else launch_variant<128, false, true, true, false, true>(p, a_mn, b_mn, grid, st);
    } else {
      if (BN == 256) launch_variant<256, false, false, true, false, true>(p, a_mn, b_mn, grid, st);
      else launch_variant<128, false, false, true, false, true>(p, a_mn, b_mn, grid, st);
    }
  } else if (tma) {
    if (g.precise) {
      if (BN == 256) launch_variant<256, false, true, true>(p, a_mn, b_mn, grid, st);
      else launch_variant<128, false, true, true>(p, a_mn, b_mn, grid, st);
    } else {
      if (BN == 256) launch_variant<256, false, false, true>(p, a_mn, b_mn, grid, st);
      else launch_variant<128, false, false, true>(p, a_mn, b_mn, grid, st);
    }
  } else {
    if (g.precise) {
      if (BN == 256) launch_variant<256, false, true, false>(p, a_mn, b_mn, grid, st);
      else launch_variant<128, false, true, false>(p, a_mn, b_mn, grid, st);
    } else {
      if (BN == 256) launch_variant<256, false, false, false>(p, a_mn, b_mn, grid, st);
      else launch_variant<128, false, false, false>(p, a_mn, b_mn, grid, st);
    }
  }
  if (cudaGetLastError() != cudaSuccess) return DION_ERR_CUDA;
  if (splits > 1) {
    const i64 total = g.M * g.N;
    int blocks = (int)((total + 255) / 256);
    if (blocks > 8 * sm_count) blocks = 8 * sm_count;
    k_splitk_reduce<<<dim3((unsigned)blocks, (unsigned)nbat), 256, 0, st>>>(part, splits, g.M, g.N, g.C, g.ldc, g.alpha, g.tri, 128, g.skip_flag,
                                                                            nbat > 1 ? g.bs2 : 0, nbat > 1 ? g.skip_stride : 0, g.alpha_dev,
                                                                            g.alpha_dev_stride);
    if (cudaGetLastError() != cudaSuccess) return DION_ERR_CUDA;
    return 2;
  }
  return 1;
}

}  // namespace dion

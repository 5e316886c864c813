// C-ABI of the Dion step library: context, argument checks, scratch layout and
// the launch sequence of one step.  All arithmetic runs in the kernels of this
// directory; the host code only validates and launches.
#include <math.h>
#include <stdlib.h>
#include <atomic>
#include <functional>
#include <mutex>
#include <new>
#include <string.h>
#include <vector>

#include "bf16_kernels.cuh"
#include "dion_common.cuh"
#include "dion_internal.h"
#include "orth_kernels.cuh"
#include "simt_gemm.cuh"
#include "umma_gemm.cuh"

using namespace dion;

namespace {

constexpr int MAX_GRAPHS = 64;             // cached step graphs per context (least recently used goes first)
constexpr i64 GRAPH_MAX_ELEMS = (i64)2048 * 2048;   // graph replay for matrices up to this many elements (launch-bound steps)
constexpr int MAX_FLAG_SLOTS = 4096;      // step slots of OS_SLOT_INTS ints each; the last MAX_GRAPHS belong to the cached graphs
constexpr int MAX_CHAIN = 64;              // matrices of one shape stepped together by dion_step_grouped
constexpr size_t GROUP_SCRATCH_BYTES = (size_t)16 << 30;  // scratch dion_step_grouped may use for that (or cfg.workspace_bytes)
constexpr int MAX_ROUNDS = 6;             // adaptive Cholesky QR rounds
constexpr float FLOOR_REL = 1e-4f;        // pivot floor relative to the column's squared norm
constexpr float GOOD_REL = 1e-4f;         // smallest relative pivot of a round that one more round can finish
// CholeskyQR2: the second round is skipped when the first round's U1 is orthonormal enough, measured as an
// estimate of |U1^T U1 - I|_F^2 (k_probe_*): done when it is <= ORTH_TAU_F^2 * r, i.e. when the deviation's
// Frobenius norm is what r entries of size ORTH_TAU_F would give.  Measured on the workloads' own panels
// (cond(P) 2-4, r 128-2048, up to 14336 rows): sqrt(estimate / r) is 5e-7 to 9e-6 after one accurate round, and the
// step's outputs then differ from the float64 rule by 3-4e-6 (Q), the same as after two rounds; warm starts
// with nearly parallel columns give 3.6e-5 and more and take the second round.
constexpr float ORTH_TAU_F = 3e-5f;
constexpr float DONE_REL = 0.9f;          // smallest relative pivot of a round whose input was already orthonormal
constexpr i64 PART_CAP_FLOATS = (i64)16 << 20;  // split-K partial sums, at most 64 MiB
constexpr double P_HALF_MIN_MNR = 4e9;          // smallest m n r whose full-rank P runs on scaled half pairs
constexpr double SOLVE_PAIR_MIN_PANEL = 3e7;    // smallest rows x r whose blocked solves run on scaled half pairs
constexpr double GRAM_PAIR_MIN_FLOPS = 2e9;     // smallest rows r^2 whose Gram matrix runs on scaled half pairs
constexpr double P_PAIR_MIN_MNR = 1.5e10;       // smallest m n r whose P = (M + G) Q runs on bf16 operand pairs first

constexpr i64 NBO_COLS = 512;  // = NBO, the outer block of the two-level Cholesky (defined below)

inline i64 align64(i64 floats) { return (floats + 63) / 64 * 64; }  // 256-byte granules

struct Layout {
  i64 P0, P1, R, Gram, Linv, Tbuf, Dinv, DinvP, part, cn_part, d, gdiag, scal, total;
  i64 Sk, SkV, SkW;         // randomized Cholesky QR: the two stacked panels [S P; P] and a solve temporary
  i64 B16, Q16, U16, R16;   // bf16-operand mode: bf16(M + G) and the bf16 copies of Q, U, R (offsets in floats)
  i64 B32;                  // fp32 mode: M + G formed once per step (0: the products form it on the fly)
  i64 Psave;                // CholeskyQR2: the panel as the product wrote it, kept for the fallback (0: none)
  i64 fb_part, fb_h, fb_n;  // fallback kernel: partial dot products (SMs x r), their sums (r), partial norms (SMs)
  i64 probe_y, probe_part;  // CholeskyQR2's orthogonality probe: U1 z (rows x NPROBE), partial U1^T (U1 z)
  i64 Bp;                   // fp32 mode, M + G in scratch: the same sum as a bf16 (hi, lo) pair (m x n x 2 bf16) for R; 0: none
  i64 Bh;                   // full rank: M + G as a scaled pair of half arrays for P (m x n x 2 halves), 0: none
  i64 pmax;                 // ... its partial maxima and the product's scale factor (like gmax)
  i64 SolveP, LfP, smax;    // blocked solves on half pairs (r > 512): pair of a rows x 512 right-hand side; pairs of a row block of
                            // the factor (512 x r) and of a diagonal inverse (512 x 512); partial maxima and scales
  i64 gmax;                 // Gram matrices on half pairs: AMAX_PARTS partial maxima of |P|, then 1 / scale^2
  i64 Qc;                   // fp32 mode, large matrices: dense fp32 copy of Q for the chain-wide recomputation of P (0: none)
  i64 S16;                  // fp32 mode: the bf16 (hi, lo) pair of the error feedback's second factor (max(m,n) x r x 2 bf16)
  i64 part_floats;
  int cn_chunks;
  i64 cn_rows;
};

}  // namespace

struct dion_ctx {
  dion_config cfg;
  int sm_count;
  float* ws;
  size_t ws_bytes;
  int* dev_ints;  // [0] status, [1] skipped, [2..] per-step flags
  int flag_cursor;
  int64_t launches;
  // per-phase profiling (off by default)
  bool prof_on;
  std::vector<cudaEvent_t> prof_pool;   // reusable events
  size_t prof_used;
  struct ProfRec { int phase; cudaEvent_t e0, e1; int64_t launches; };
  std::vector<ProfRec> prof_recs;
  // second stream for work that can run beside the serial Cholesky chain, and its fork/join events
  bool form_sum = true;   // fp32 mode may keep M + G in scratch (off for the fixed-scratch entry point)
  cudaStream_t side = nullptr;
  cudaEvent_t side_ev[32] = {};
  int side_cursor = 0;
  // Graph replay of launch-bound steps: the launch chain of dion_step on a small matrix is captured once per
  // (descriptor) into a CUDA graph and replayed; the learning rate reaches it through a device scalar.
  struct GraphEntry {
    dion_matrix key;
    cudaGraphExec_t exec;
    int64_t launches;
    int index;            // its state slot and scalar
    uint64_t last_use;
  };
  std::vector<GraphEntry> graphs;
  bool graphs_on = false;
  bool chain_batch = true;          // tensor-engine products of a grouped chain in one launch over its matrices
  cudaStream_t cap = nullptr;       // the stream the chains are captured on (never the caller's: it may be the legacy stream)
  float* graph_scalars = nullptr;   // MAX_GRAPHS device floats
  uint64_t graph_clock = 0;
};

namespace {

void colnorm_plan(i64 rows, i64 r, int sm, int* chunks, i64* rows_per) {
  const i64 col_blocks = (r + 127) / 128;
  i64 want = (4 * (i64)sm + col_blocks - 1) / col_blocks;
  if (want < 1) want = 1;
  i64 per = (rows + want - 1) / want;
  if (per < 32) per = 32;
  *rows_per = per;
  *chunks = (int)((rows + per - 1) / per);
}

// fp32 mode on the tensor engine: M + G is formed once per step in scratch, as fp32 (4 bytes per element) and as a
// bf16 (hi, lo) pair (4 bytes), and P, R and the error feedback read those.  Forming it inside the two products
// costs their converter warps a second tile and keeps them on three TF32 MMAs per K step; with the pair in
// memory the products take three bf16 MMAs (half the tensor time) and read 4 bytes per element instead of 8, so the
// extra pass pays down to rank fraction 1/64 (measured: 32768^2 at r = 512 22.0 -> 15.9 ms, 16384^2 at r = 256
// 3.4 -> 3.0 ms); below that the step is HBM bound either way and the on-the-fly form moves fewer bytes.
bool sum_in_scratch(const dion_ctx* c, i64 m, i64 n, i64 r) {
  const i64 sd = (m < n) ? m : n;
  return c->form_sum && c->cfg.precision == DION_PREC_FP32 && c->cfg.engine != DION_ENGINE_SIMT &&
         m % 4 == 0 && n % 4 == 0 && m >= 128 && n >= 128 && r >= 64 && 64 * r >= sd;
}

// Above rank fraction 1/4 (the adaptive rounds: ill-conditioned panels) P = (M + G) Q needs its 22 significant
// bits.  On large matrices it takes them from scaled pairs of IEEE half arrays (three kind::f16 MMAs per K step,
// split accumulators) instead of the 3xTF32 split with four kind::tf32 ones: M + G is scaled by a power of two
// found on the device, Q (unit-norm columns) by 2^13.
int resolve_orth(const dion_ctx* c, i64 r, i64 short_dim);
bool p_on_half_pairs(const dion_ctx* c, i64 m, i64 n, i64 r) {
  return c->cfg.precision == DION_PREC_FP32 && c->cfg.engine != DION_ENGINE_SIMT && m % 8 == 0 && n % 8 == 0 && r % 8 == 0 &&
         (double)m * (double)n * (double)r >= P_HALF_MIN_MNR && resolve_orth(c, r, (m < n) ? m : n) == DION_ORTH_SHIFTED3;
}

// A step whose orthonormalization may resolve to CholeskyQR2 keeps the panel for the device-side fallback.
bool may_fallback(const dion_ctx* c, i64 m, i64 n, i64 r) {
  const i64 sd = (m < n) ? m : n;
  const int o = c->cfg.orth;
  return o == DION_ORTH_CHOLQR2 || ((o == DION_ORTH_AUTO || o == DION_ORTH_RCQR) && 4 * r <= sd);
}

Layout make_layout(const dion_ctx* c, i64 m, i64 n, i64 r) {
  Layout L;
  const i64 big = (m > n) ? m : n;
  i64 o = 0;
  L.P0 = o; o += align64(big * r);
  L.P1 = o; o += align64(big * r);
  L.R = o; o += align64(big * r);
  L.Gram = o; o += align64(r * r);
  L.Linv = o; o += align64(r * r);
  L.Tbuf = o; o += align64(r * r);
  L.Dinv = o; o += align64(((r + NB - 1) / NB) * (i64)NB * NB);
  L.DinvP = o; o += align64(((r + NB - 1) / NB) * (i64)NB * NB);
  // split-K partials: the largest plain-store product of a step is max(m,n) x r
  i64 pf = 4 * (i64)c->sm_count * 64 * 64;
  if (pf > PART_CAP_FLOATS) pf = PART_CAP_FLOATS;
  L.part_floats = pf;
  L.part = o; o += align64(pf);
  colnorm_plan(big, r, c->sm_count, &L.cn_chunks, &L.cn_rows);
  L.cn_part = o; o += align64((i64)(L.cn_chunks + 1) * r);
  L.d = o; o += align64(r);
  L.gdiag = o; o += align64(r);
  L.scal = o; o += 64;
  L.Sk = L.SkV = 0;
  L.SkW = 0;
  if (c->cfg.orth == DION_ORTH_RCQR) {
    // two (sketch rows + panel rows) x r buffers for the rounds on the stacked panel [S P; P], and the
    // 512-column temporary of their blocked solves
    L.Sk = o; o += align64((2 * r + big) * r);
    L.SkV = o; o += align64((2 * r + big) * r);
    L.SkW = o; o += align64((2 * r + big) * NBO_COLS);
  }
  L.B16 = L.Q16 = L.U16 = L.R16 = 0;
  if (c->cfg.precision == DION_PREC_BF16_OPERANDS) {
    L.B16 = o; o += align64((m * n + 1) / 2);
    L.Q16 = o; o += align64((big * r + 1) / 2);
    L.U16 = o; o += align64((big * r + 1) / 2);
    L.R16 = o; o += align64((big * r + 1) / 2);
  }
  L.B32 = L.Bp = 0;
  if (sum_in_scratch(c, m, n, r)) {
    L.B32 = o; o += align64(m * n);
    if (m % 8 == 0 && n % 8 == 0 && r % 8 == 0) { L.Bp = o; o += align64(m * n); }
  }
  L.Psave = L.fb_part = L.fb_h = L.fb_n = 0;
  L.gmax = o; o += align64(AMAX_PARTS + 64);
  L.SolveP = L.LfP = L.smax = 0;
  if (r > NBO_COLS && (double)big * (double)r >= SOLVE_PAIR_MIN_PANEL) {
    L.SolveP = o; o += align64(big * NBO_COLS);
    L.LfP = o; o += align64(NBO_COLS * r + NBO_COLS * NBO_COLS);
    L.smax = o; o += align64(3 * (AMAX_PARTS + 64));
  }
  L.Bh = L.pmax = 0;
  if (L.Bp > 0 && p_on_half_pairs(c, m, n, r)) {
    L.Bh = o; o += align64(m * n);
    L.pmax = o; o += align64(AMAX_PARTS + 64);
  }
  L.Qc = 0;
  if (L.Bp > 0 && (double)m * (double)n * (double)r >= P_PAIR_MIN_MNR) { L.Qc = o; o += align64(big * r); }
  L.S16 = o; o += align64(big * r);
  L.probe_y = o; o += align64(big * NPROBE);
  L.probe_part = o; o += align64((i64)(L.cn_chunks + 1) * r * NPROBE);
  if (may_fallback(c, m, n, r)) {
    L.Psave = o; o += align64(big * r);
    L.fb_part = o; o += align64((i64)c->sm_count * r);
    L.fb_h = o; o += align64(r);
    L.fb_n = o; o += align64(c->sm_count);
  }
  L.total = o;
  return L;
}

void graphs_clear(dion_ctx* c);

int ensure_ws(dion_ctx* c, size_t bytes) {
  if (bytes <= c->ws_bytes) return DION_OK;
  if (c->ws != nullptr) {
    if (cudaDeviceSynchronize() != cudaSuccess) return DION_ERR_CUDA;
    graphs_clear(c);      // they point into the old scratch
    cudaFree(c->ws);
    c->ws = nullptr;
    c->ws_bytes = 0;
  }
  void* p = nullptr;
  if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return DION_ERR_NOMEM; }
  c->ws = (float*)p;
  c->ws_bytes = bytes;
  return DION_OK;
}

#define DION_CHECK_LAUNCH(ctx)                                   \
  do {                                                           \
    (ctx)->launches++;                                           \
    if (cudaGetLastError() != cudaSuccess) return DION_ERR_CUDA; \
  } while (0)
#define DION_TRY(expr)              \
  do {                              \
    const int rc_ = (expr);         \
    if (rc_ != DION_OK) return rc_; \
  } while (0)

GemmArgs gemm_args() {
  GemmArgs g;
  memset(&g, 0, sizeof(g));
  g.alpha = 1.f;
  g.batch = 1;
  g.batch2 = 1;
  g.splits = 1;
  return g;
}

// Launch with programmatic stream serialization (see pdl_enter in the kernels).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// Launches one product on the fp32 FMA engine.
int launch_gemm_simt(dion_ctx* c, GemmArgs g, cudaStream_t st, float* part, i64 part_floats,
                     bool force64) {
  if (g.M <= 0 || g.N <= 0) return DION_OK;
  const i64 t128 = ((g.M + 127) / 128) * ((g.N + 127) / 128) * g.batch * (g.batch2 > 1 ? g.batch2 : 1);
  const bool use128 = !force64 && t128 >= c->sm_count;
  const int BMN = use128 ? 128 : 64;
  const i64 gm = (g.M + BMN - 1) / BMN, gn = (g.N + BMN - 1) / BMN;
  int splits = 1;
  if (!use128 && !force64 && g.epi == EPI_STORE && g.batch == 1 && g.batch2 <= 1 && part != nullptr && g.alpha_dev == nullptr) {
    const i64 tiles = gm * gn;
    i64 want = (2 * (i64)c->sm_count + tiles - 1) / tiles;
    const i64 kmax = g.K / 128;
    if (want > kmax) want = kmax;
    if (want > 64) want = 64;
    while (want > 1 && want * g.M * g.N > part_floats) --want;
    if (want > 1) splits = (int)want;
  }
  g.splits = splits;
  g.part = part;
  if (gm > 65535) return DION_ERR_UNSUPPORTED;
  if (g.batch2 < 1) g.batch2 = 1;
  if (splits > 1 && g.batch2 > 1) return DION_ERR_INVALID;
  dim3 grid((unsigned)gn, (unsigned)gm, (unsigned)(splits > 1 ? splits : g.batch * g.batch2));
  if (use128) launch_pdl(k_gemm_simt<128, 128, 8, 8, 8>, grid, dim3(256), 0, st, g);
  else launch_pdl(k_gemm_simt<64, 64, 16, 4, 4>, grid, dim3(256), 0, st, g);
  DION_CHECK_LAUNCH(c);
  if (splits > 1) {
    const i64 total = g.M * g.N;
    int blocks = (int)((total + 255) / 256);
    if (blocks > 8 * c->sm_count) blocks = 8 * c->sm_count;
    launch_pdl(k_splitk_reduce, dim3((unsigned)(blocks)), dim3(256), 0, st, part, splits, g.M, g.N, g.C, g.ldc, g.alpha, g.tri, BMN, g.skip_flag, (i64)0, (i64)0, (const float*)nullptr, (i64)0);
    DION_CHECK_LAUNCH(c);
  }
  return DION_OK;
}

cudaEvent_t prof_event(dion_ctx* c) {
  if (c->prof_used == c->prof_pool.size()) {
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    c->prof_pool.push_back(e);
  }
  return c->prof_pool[c->prof_used++];
}

// Brackets one phase of a step with events on the step's stream when profiling is on.
struct PhaseScope {
  dion_ctx* c; cudaStream_t st; int phase; cudaEvent_t e0; int64_t l0;
  PhaseScope(dion_ctx* c_, cudaStream_t st_, int phase_) : c(c_), st(st_), phase(phase_), e0(nullptr), l0(c_->launches) {
    if (c->prof_on && phase >= 0) { e0 = prof_event(c); if (e0) cudaEventRecord(e0, st); }
  }
  ~PhaseScope() {
    if (c->prof_on && e0) {
      cudaEvent_t e1 = prof_event(c);
      if (e1) { cudaEventRecord(e1, st); c->prof_recs.push_back({phase, e0, e1, c->launches - l0}); }
    }
  }
};

// One launch chain works on `nb` matrices of identical (m, n, r) at a time (nb = 1 for
// dion_step): the large products are launched per matrix, the small kernels of the
// factorization once for all of them (one block or batch entry per matrix).  Matrix b
// uses the scratch slice that starts b * wstride floats after `ws` and the state slot
// b * OS_SLOT_INTS ints after `os`.
struct StepCtx {
  dion_ctx* c;
  cudaStream_t st;
  float* ws;
  Layout L;
  int nb;
  i64 wstride;
  int* os;    // first device state slot (OS_* ints)
  int* flag;  // = os + OS_FAIL: the step must not write its outputs
  bool tensor;  // tensor-core engine allowed for this matrix
  bool in_orth; // inside the orthonormalization (for the profiling phases)
  const dion_matrix* const* list = nullptr;   // the matrices of the chain (sketch pointers of the RCQR mode)
  i64 wt_off = -1;        // >= 0: scratch offset of the blocked solves' rows x 512 temporary (default: the R panel)
  bool no_split = false;  // launches on the side stream: the split-K scratch belongs to the main stream
  bool quiet_fail = false;  // a failed pivot only sets the step's fail flag: the fallback kernel follows
  const std::function<int()>* redo_p = nullptr;   // the panel came from the fast product: recomputes it accurately
                                                  // (skipped on the device for matrices whose OS_DONE is set)
  float* W(int b, i64 off) const { return ws + (i64)b * wstride + off; }
  int* OS(int b) const { return os + (i64)b * OS_SLOT_INTS; }
};

// Engine dispatch: tensor cores when the product qualifies, else fp32 FMA.
// `b`: the matrix of the batch the product belongs to (selects its split-K scratch).
int launch_gemm(StepCtx& s, const GemmArgs& g, int b = 0, bool force64 = false) {
  if (s.tensor && !force64) {
    PhaseScope ps(s.c, s.st, s.in_orth ? DION_PHASE_ORTH_GEMM : -1);
    // bf16 operands are for the four large contractions only: the Gram matrices, factors and
    // solves of the orthonormalization keep fp32 accuracy in every mode
    const int prec = s.in_orth ? DION_PREC_FP32 : s.c->cfg.precision;
    const int rc = umma_try_launch(g, prec, s.c->sm_count, s.no_split ? nullptr : s.W(b, s.L.part), s.L.part_floats,
                                   s.c->dev_ints, s.st);
    if (rc > 0) { s.c->launches += rc; return DION_OK; }
    if (rc < 0) return rc;
    if (s.c->cfg.engine == DION_ENGINE_TENSOR) return DION_ERR_UNSUPPORTED;
  }
  if (g.ab16) return DION_ERR_UNSUPPORTED;   // bf16 arrays are read by the tensor engine only
  return launch_gemm_simt(s.c, g, s.st, s.no_split ? nullptr : s.W(b, s.L.part), s.L.part_floats, force64);
}

// Shifts the workspace-resident operands of a product to matrix b of the batch.
GemmArgs for_matrix(const StepCtx& s, GemmArgs g, int b, bool a_ws, bool b_ws, bool c_ws) {
  const i64 o = (i64)b * s.wstride;
  if (a_ws) g.A += o;
  if (b_ws) g.B += o;
  if (c_ws) g.C += o;
  if (a_ws && g.A16lo != nullptr) g.A16lo = (const char*)g.A16lo + 4 * o;
  if (b_ws && g.B16lo != nullptr) g.B16lo = (const char*)g.B16lo + 4 * o;
  if (g.alpha_dev != nullptr) g.alpha_dev += (i64)b * g.alpha_dev_stride;
  if (g.skip_flag != nullptr) g.skip_flag += (i64)b * OS_SLOT_INTS;
  return g;
}

void over_batch(const StepCtx& s, GemmArgs& g);

// One product per matrix of the chain, operands and output in the scratch slices (c2_ws: the second epilogue
// operand too).  The tensor engine takes all matrices in one launch when the product qualifies (its work list
// then runs over (matrix, tile) pairs, which also fills the tail of one matrix's tiles with the next one's);
// otherwise one launch per matrix.
int launch_gemm_chain(StepCtx& s, const GemmArgs& g, bool c2_ws = false) {
  if (s.nb > 1 && s.tensor && s.c->chain_batch) {
    GemmArgs gb = g;
    over_batch(s, gb);
    gb.c2_batched = c2_ws ? 1 : 0;
    PhaseScope ps(s.c, s.st, s.in_orth ? DION_PHASE_ORTH_GEMM : -1);
    const int prec = s.in_orth ? DION_PREC_FP32 : s.c->cfg.precision;
    const int rc = umma_try_launch(gb, prec, s.c->sm_count, s.no_split ? nullptr : s.W(0, s.L.part), s.L.part_floats,
                                   s.c->dev_ints, s.st);
    if (rc > 0) { s.c->launches += rc; return DION_OK; }
    if (rc < 0) return rc;
  }
  for (int m = 0; m < s.nb; ++m) {
    GemmArgs gm = for_matrix(s, g, m, true, true, true);
    if (c2_ws) gm.C2 = (const float*)gm.C2 + (i64)m * s.wstride;
    DION_TRY(launch_gemm(s, gm, m));
  }
  return DION_OK;
}

// The same product on every matrix of the chain, given as one GemmArgs per matrix (as the per-matrix launch would
// take them).  When the tensor engine can run them as ONE launch -- identical shapes and strides, operands in the
// scratch slices (so that one 3-D tensor map covers them), outputs anywhere (a pointer table) -- it does: the work
// list then runs over (matrix, tile) pairs and the last wave of one matrix is filled with the next one's tiles.
// Every element is computed by the same sequence of operations either way.
int launch_gemm_group(StepCtx& s, const std::vector<GemmArgs>& v) {
  const int nb = (int)v.size();
  bool one = nb > 1 && nb <= GEMM_TAB_MAX && s.tensor && s.c->chain_batch;
  const GemmArgs& a = v[0];
  bool c_strided = true, c2_strided = true;
  const i64 wb = s.wstride * 4;   // bytes between scratch slices
  auto at_stride = [&](const void* p0, const void* pb, int b) {
    return (p0 == nullptr && pb == nullptr) ||
           (p0 != nullptr && pb != nullptr && (const char*)pb - (const char*)p0 == (ptrdiff_t)((i64)b * wb));
  };
  for (int b = 1; b < nb && one; ++b) {
    const GemmArgs& g = v[b];
    one = g.M == a.M && g.N == a.N && g.K == a.K && g.a_si == a.a_si && g.a_sk == a.a_sk && g.a2_si == a.a2_si &&
          g.a2_sk == a.a2_sk && g.a2_mode == a.a2_mode && g.b_sk == a.b_sk && g.b_sn == a.b_sn && g.ldc == a.ldc &&
          g.epi == a.epi && g.ldc2 == a.ldc2 && g.c2_mode == a.c2_mode && g.alpha == a.alpha &&
          (g.alpha_dev == a.alpha_dev || at_stride(a.alpha_dev, g.alpha_dev, b)) &&
          g.batch == 1 && a.batch == 1 && g.tri == a.tri && g.klimit == a.klimit && g.precise == a.precise &&
          g.ab16 == a.ab16 && g.f16 == a.f16 && g.tf32x1 == a.tf32x1 && at_stride(a.A, g.A, b) && at_stride(a.B, g.B, b) &&
          at_stride(a.A2, g.A2, b) && at_stride(a.A16lo, g.A16lo, b) && at_stride(a.B16lo, g.B16lo, b) &&
          ((a.skip_flag == nullptr && g.skip_flag == nullptr) ||
           (a.skip_flag != nullptr && g.skip_flag == a.skip_flag + (i64)b * OS_SLOT_INTS));
    c_strided = c_strided && at_stride(a.C, g.C, b);
    c2_strided = c2_strided && at_stride(a.C2, g.C2, b);
  }
  if (one && !c_strided && a.epi == EPI_STORE) one = false;   // (a plain store may split K: its reduction wants one stride)
  if (one) {
    GemmArgs gb = a;
    over_batch(s, gb);
    if (nb > 1 && v[1].alpha_dev != a.alpha_dev) gb.alpha_dev_stride = s.wstride;     // a scale per matrix, in its scratch slice
    float* ctab[GEMM_TAB_MAX];
    const void* c2tab[GEMM_TAB_MAX];
    for (int b = 0; b < nb; ++b) { ctab[b] = v[b].C; c2tab[b] = v[b].C2; }
    if (!c_strided) gb.c_tab = ctab;
    if (a.C2 != nullptr) {
      if (c2_strided && a.c2_mode == ADD_F32) gb.c2_batched = 1;
      else gb.c2_tab = c2tab;
    }
    PhaseScope ps(s.c, s.st, s.in_orth ? DION_PHASE_ORTH_GEMM : -1);
    const int prec = s.in_orth ? DION_PREC_FP32 : s.c->cfg.precision;
    const int rc = umma_try_launch(gb, prec, s.c->sm_count, s.no_split ? nullptr : s.W(0, s.L.part), s.L.part_floats,
                                   s.c->dev_ints, s.st);
    if (rc > 0) { s.c->launches += rc; return DION_OK; }
    if (rc < 0) return rc;
  }
  for (int b = 0; b < nb; ++b) DION_TRY(launch_gemm(s, v[b], b));
  return DION_OK;
}

// One-time opt-in to the dynamic shared memory of the kernels that need more than 48 KB.
int configure_kernels() {
  if (umma_configure() != DION_OK) return DION_ERR_CUDA;
  if (cudaFuncSetAttribute(k_probe_y4, cudaFuncAttributeMaxDynamicSharedMemorySize, PY_SMEM) != cudaSuccess ||
      cudaFuncSetAttribute(k_chol_step, cudaFuncAttributeMaxDynamicSharedMemorySize, CHOL_STEP_SMEM) != cudaSuccess ||
      cudaFuncSetAttribute(k_tiny_cholqr2, cudaFuncAttributeMaxDynamicSharedMemorySize, tiny_cholqr2_smem(TINY_MAX_ROWS)) != cudaSuccess) {
    cudaGetLastError();
    return DION_ERR_CUDA;
  }
  return DION_OK;
}

constexpr i64 NBO = NBO_COLS;  // outer block of the two-level Cholesky

int grid_for(const dion_ctx* c, i64 total) {
  i64 blocks = (total + 255) / 256;
  if (blocks > 8 * (i64)c->sm_count) blocks = 8 * (i64)c->sm_count;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

// Marks a small (FMA-engine) product as batched over the nb matrices of the chain.
void over_batch(const StepCtx& s, GemmArgs& g) {
  g.batch2 = s.nb;
  g.bs2 = s.wstride;
  g.skip_stride = OS_SLOT_INTS;
}

// Inverse of a lower-triangular matrix by doubling, on the diagonal square [o, o+sz):
// [[L11,0],[L21,L22]]^-1 = [[X11,0],[-X22 L21 X11, X22]], for block sizes b_from, 2 b_from, ...
// while b < sz.  The diagonal blocks of size b_from of Linv must already hold their inverses.
// Offsets are relative to each matrix's scratch slice.
int trtri_levels(StepCtx& s, i64 r, i64 o, i64 sz, i64 b_from, const int* skip, int precise) {
  const float* Gm = s.ws + s.L.Gram;
  float* Linv = s.ws + s.L.Linv;
  float* Tbuf = s.ws + s.L.Tbuf;
  for (i64 b = b_from; b < sz; b *= 2) {
    const i64 nfull = sz / (2 * b);
    const i64 tail0 = nfull * 2 * b;
    const i64 b2_tail = (sz - tail0 > b) ? (sz - tail0 - b) : 0;
    for (int pass = 0; pass < 2; ++pass) {
      const i64 base = o + ((pass == 0) ? 0 : tail0);
      const i64 rows = (pass == 0) ? b : b2_tail;
      const int batch = (pass == 0) ? (int)nfull : 1;
      if (rows <= 0 || batch <= 0) continue;
      const i64 off21 = (base + b) * r + base, off11 = base * r + base, off22 = (base + b) * r + (base + b);
      const i64 bs = 2 * b * (r + 1);
      const bool big = b >= NBO;   // large blocks: one launch per pair and matrix, tensor cores where they qualify
      const int launches = big ? batch : 1;
      for (int q = 0; q < launches; ++q) {
        const i64 sh = big ? (i64)q * bs : 0;
        GemmArgs g1 = gemm_args();  // T = L21 * X11
        g1.M = rows; g1.N = b; g1.K = b;
        g1.A = Gm + off21 + sh; g1.a_si = r; g1.a_sk = 1;
        g1.B = Linv + off11 + sh; g1.b_sk = r; g1.b_sn = 1;
        g1.C = Tbuf + off21 + sh; g1.ldc = r; g1.epi = EPI_STORE; g1.skip_flag = skip; g1.precise = precise;
        GemmArgs g2 = gemm_args();  // X21 = -X22 * T
        g2.M = rows; g2.N = b; g2.K = rows;
        g2.A = Linv + off22 + sh; g2.a_si = r; g2.a_sk = 1;
        g2.B = Tbuf + off21 + sh; g2.b_sk = r; g2.b_sn = 1;
        g2.C = Linv + off21 + sh; g2.ldc = r; g2.epi = EPI_STORE; g2.alpha = -1.f; g2.skip_flag = skip; g2.precise = precise;
        if (big) {
          DION_TRY(launch_gemm_chain(s, g1));
          DION_TRY(launch_gemm_chain(s, g2));
        } else {
          g1.batch = batch; g1.bsA = bs; g1.bsB = bs; g1.bsC = bs; over_batch(s, g1);
          g2.batch = batch; g2.bsA = bs; g2.bsB = bs; g2.bsC = bs; over_batch(s, g2);
          DION_TRY(launch_gemm_simt(s.c, g1, s.st, nullptr, 0, false));
          DION_TRY(launch_gemm_simt(s.c, g2, s.st, nullptr, 0, false));
        }
      }
    }
  }
  return DION_OK;
}

// Cholesky of the diagonal square [o, o+sz) of each Gram matrix (sz <= NBO), right-looking with
// 64-wide blocks on the FMA engine, followed by the inverse of that square's factor into Linv.
// How a Cholesky-QR round runs.
enum : int {
  RM_PLAIN = 0,     // no device-side control
  RM_ADAPTIVE = 1,  // deflating pivots, skipped once the panel is done, split-accumulator products, round statistics
  RM_FIRST = 2,     // first round of CholeskyQR2: plain control, split-accumulator products
  RM_CHECKED = 3,   // second round of CholeskyQR2: the first round's result is measured first (orthogonality probe);
                    // if it is orthonormal to ORTH_TAU_F the whole round is skipped (Pout = Pin)
  RM_REDO = 4       // first round once more, on the panel recomputed with the accurate product: skipped on the device
                    // when the round on the fast panel already passed the probe; split-accumulator products
};
inline bool rm_skips(int mode) { return mode == RM_ADAPTIVE || mode == RM_CHECKED || mode == RM_REDO; }
inline bool rm_precise(int mode) { return mode == RM_ADAPTIVE || mode == RM_FIRST || mode == RM_REDO; }

int potrf_inner(StepCtx& s, i64 r, i64 o, i64 sz, int mode) {
  const bool adaptive = rm_skips(mode);
  dion_ctx* c = s.c;
  float* Gm = s.ws + s.L.Gram;
  float* Dinv = s.ws + s.L.Dinv;
  float* DinvP = s.ws + s.L.DinvP;
  float* Linv = s.ws + s.L.Linv;
  float* Tbuf = s.ws + s.L.Tbuf;
  const float* gdiag = s.ws + s.L.gdiag;
  int* status = s.quiet_fail ? nullptr : c->dev_ints;
  const int* skip = adaptive ? (s.os + OS_DONE) : nullptr;
  const float floor_rel = (mode == RM_ADAPTIVE) ? FLOOR_REL : 0.f;
  const int nblk = (int)((sz + NB - 1) / NB);
  {
    const int jb = (int)((sz < NB) ? sz : NB);
    launch_pdl(k_potrf_diag, dim3((unsigned)s.nb), dim3(256), 0, s.st, Gm + o * r + o, r, jb, Dinv + (o / NB) * (NB * NB),
               DinvP + (o / NB) * (NB * NB), gdiag + o, floor_rel, s.os, adaptive ? 1 : 0, status, s.wstride);
    DION_CHECK_LAUNCH(c);
  }
  // one launch per block column: panel, trailing update and the next diagonal block; behind them the CTAs
  // that add one term to every unfinished block row of the inverse of the square's factor (j blocks in each
  // of the rows j .. nblk-1), off the critical path
  for (int j = 0; j + 1 < nblk; ++j) {
    const int nt = nblk - 1 - j;
    const int extra = (nblk - j) * j;
    dim3 grid((unsigned)(nt * (nt + 1) / 2 + extra), (unsigned)s.nb);
    launch_pdl(k_chol_step, grid, dim3(256), CHOL_STEP_SMEM, s.st, Gm, r, o, sz, j, Dinv, DinvP, Tbuf, Linv, gdiag, floor_rel,
               s.os, adaptive ? 1 : 0, status, s.wstride);
    DION_CHECK_LAUNCH(c);
  }
  {
    // last block row of the inverse, the factor's blocks into the Gram buffer, diagonal inverses into Linv
    dim3 grid((unsigned)(nblk - 1 + grid_for(c, sz * sz)), (unsigned)s.nb);
    launch_pdl(k_inv_finish, grid, dim3(256), INV_FINISH_SMEM, s.st, (const float*)Tbuf, Gm, Linv, r, o, sz, (const float*)Dinv, skip,
               s.wstride);
    DION_CHECK_LAUNCH(c);
  }
  return DION_OK;
}

// Two-level blocked Cholesky of each r x r Gram matrix (lower) and the full inverse of its
// factor into Linv.  Outer blocks of 512 columns: the diagonal square is factored and
// inverted by potrf_inner, the panel below it is multiplied by that inverse and the
// trailing matrix is updated with one rank-512 product (tensor cores where it qualifies).
int potrf_trtri(StepCtx& s, i64 r, int mode, bool full_inverse,
                const std::function<int(i64, i64)>* after_block = nullptr) {
  const bool adaptive = rm_skips(mode);
  dion_ctx* c = s.c;
  float* Gm = s.ws + s.L.Gram;
  float* Linv = s.ws + s.L.Linv;
  float* Tbuf = s.ws + s.L.Tbuf;
  const int* skip = adaptive ? (s.os + OS_DONE) : nullptr;
  const int precise = rm_precise(mode) ? 1 : 0;
  if (r > NBO && full_inverse) {
    // everything outside the diagonal squares starts at zero (the product U = P Linv^T reads whole tiles)
    for (int m = 0; m < s.nb; ++m)
      if (cudaMemsetAsync(s.W(m, s.L.Linv), 0, sizeof(float) * (size_t)r * (size_t)r, s.st) != cudaSuccess) return DION_ERR_CUDA;
  }
  for (i64 J0 = 0; J0 < r; J0 += NBO) {
    const i64 sz = (r - J0 < NBO) ? (r - J0) : NBO;
    DION_TRY(potrf_inner(s, r, J0, sz, mode));
    if (after_block != nullptr) DION_TRY((*after_block)(J0, sz));   // block column J of the factor and its inverse are final
    const i64 rem = r - J0 - sz;
    if (rem > 0) {
      float* panel = Gm + (J0 + sz) * r + J0;
      float* ptmp = Tbuf + (J0 + sz) * r + J0;
      GemmArgs g = gemm_args();  // Lpanel = panel * Linv_JJ^T (out of place, then copied back)
      g.M = rem; g.N = sz; g.K = sz;
      g.A = panel; g.a_si = r; g.a_sk = 1;
      g.B = Linv + J0 * r + J0; g.b_sk = 1; g.b_sn = r; g.klimit = 1;
      g.C = ptmp; g.ldc = r; g.epi = EPI_STORE; g.skip_flag = skip; g.precise = precise;
      DION_TRY(launch_gemm_chain(s, g));
      // With the solves on the second stream, the copy of Lpanel into the Gram buffer goes there too: its
      // only readers are the solves of later block columns (queued behind it on that stream); the trailing
      // update reads the temporary, so the copy leaves the serial chain.
      const bool side_copy = after_block != nullptr && c->side != nullptr;
      {
        cudaStream_t cst = s.st;
        if (side_copy) {
          cudaEvent_t e = c->side_ev[c->side_cursor];
          c->side_cursor = (c->side_cursor + 1) % 32;
          if (cudaEventRecord(e, s.st) != cudaSuccess || cudaStreamWaitEvent(c->side, e, 0) != cudaSuccess) return DION_ERR_CUDA;
          cst = c->side;
        }
        dim3 grid((unsigned)grid_for(c, rem * sz), (unsigned)s.nb);
        launch_pdl(k_copy_block, grid, dim3(256), 0, cst, ptmp, r, panel, r, rem, sz, skip, s.wstride);
        DION_CHECK_LAUNCH(c);
      }
      const float* lp = side_copy ? ptmp : panel;
      GemmArgs t = gemm_args();  // A22 -= Lpanel * Lpanel^T (lower tiles)
      t.M = rem; t.N = rem; t.K = sz;
      t.A = lp; t.a_si = r; t.a_sk = 1;
      t.B = lp; t.b_sk = 1; t.b_sn = r;
      t.C = Gm + (J0 + sz) * r + (J0 + sz); t.ldc = r; t.epi = EPI_SUB; t.tri = TRI_LOWER; t.skip_flag = skip;
      t.precise = precise;
      DION_TRY(launch_gemm_chain(s, t));
    }
  }
  if (r > NBO && full_inverse) DION_TRY(trtri_levels(s, r, 0, r, NBO, skip, precise));
  return DION_OK;
}

// The orthogonality probe on the rows x r panels at `off` (two passes over the panel instead of its Gram matrix).
// phase: PROBE_CHECK the check of CholeskyQR2's first round; PROBE_FAST the same after a round on a panel from the
// fast product (decides whether the panel is recomputed; counts nothing); PROBE_AFTER_REDO the check that follows a
// possible recomputation (a panel that passed PROBE_FAST is not measured again).
int probe(StepCtx& s, i64 off, i64 rows, i64 r, int phase) {
  dion_ctx* c = s.c;
  int chunks; i64 per;
  colnorm_plan(rows, r, c->sm_count, &chunks, &per);
  const int* keep = (phase == PROBE_AFTER_REDO) ? (const int*)(s.os + OS_DONE) : nullptr;
  if (r % 4 == 0 && r >= 128) {
    i64 blocks = (rows + 31) / 32;          // a block of 8 warps takes 32 rows at a time
    if (blocks > 2 * (i64)c->sm_count) blocks = 2 * (i64)c->sm_count;
    launch_pdl(k_probe_y4, dim3((unsigned)blocks, (unsigned)s.nb), dim3(256), (size_t)PY_SMEM, s.st, (const float*)(s.ws + off), r, rows, r,
               s.ws + s.L.probe_y, s.wstride, keep);
  } else {
    launch_pdl(k_probe_y, dim3((unsigned)grid_for(c, rows * 32), (unsigned)s.nb), dim3(256), 0, s.st, (const float*)(s.ws + off), r,
               rows, r, s.ws + s.L.probe_y, s.wstride, keep);
  }
  DION_CHECK_LAUNCH(c);
  if (r % 4 == 0)
    launch_pdl(k_probe_w4, dim3((unsigned)((r / 4 + 127) / 128), (unsigned)chunks, (unsigned)s.nb), dim3(128), 0, s.st,
               (const float*)(s.ws + off), r, rows, r, per, (const float*)(s.ws + s.L.probe_y), s.ws + s.L.probe_part, s.wstride, keep);
  else
    launch_pdl(k_probe_w, dim3((unsigned)((r + 127) / 128), (unsigned)chunks, (unsigned)s.nb), dim3(128), 0, s.st,
               (const float*)(s.ws + off), r, rows, r, per, (const float*)(s.ws + s.L.probe_y), s.ws + s.L.probe_part, s.wstride, keep);
  DION_CHECK_LAUNCH(c);
  launch_pdl(k_probe_decide, dim3((unsigned)s.nb), dim3(r >= 128 ? 1024 : 256), 0, s.st, (const float*)(s.ws + s.L.probe_part), chunks, r, s.os,
             ORTH_TAU_F, c->dev_ints + 2, s.wstride, phase);
  DION_CHECK_LAUNCH(c);
  return DION_OK;
}

// Tall panels whose blocked triangular solves run on scaled half pairs.
// (where the solves are what the round waits for: CholeskyQR2 on large panels.  In the adaptive rounds they run
// beside the serial chain, and on the panels of the 8B list the extra passes for scales and pairs cost what the
// cheaper products save: measured, 42.1 -> 44.1 ms there, 48.1 -> 42.8 ms on the large squares.)
bool solve_on_pairs(const StepCtx& s, i64 rows, i64 r, int mode) {
  return s.tensor && s.nb <= GEMM_TAB_MAX && mode != RM_ADAPTIVE && rows % 8 == 0 && r % 8 == 0 &&
         (double)rows * (double)r >= SOLVE_PAIR_MIN_PANEL;
}

// Tall panels whose Gram matrix runs on scaled half pairs (the rule looks at the shape alone).
bool gram_on_pairs(const StepCtx& s, i64 rows, i64 r) {
  return s.tensor && rows % 8 == 0 && r % 8 == 0 && r >= 128 &&
         (double)rows * (double)r * (double)r >= GRAM_PAIR_MIN_FLOPS;      // (in either precision mode)
}

// One Cholesky-QR round on every matrix of the chain: Pout = Pin * chol(Pin^T Pin)^-T.
// rows x r panels, ld = r; pin_off / pout_off are offsets in the scratch slice.
// adaptive: columns with negligible pivots are deflated, the round is skipped (Pout = Pin)
// once the panel is orthonormal, and the round statistics are evaluated at the end.
int cholqr_round(StepCtx& s, i64 pin_off, i64 pout_off, i64 rows, i64 r, int mode, i64 gram_rows = 0,
                 bool passthrough = true, int probe_phase = PROBE_CHECK) {
  // passthrough = false: a skipped round leaves Pout untouched (the caller keeps using Pin)
  // gram_rows > 0: the Gram matrix is formed from the first gram_rows rows only (a sketch stacked on
  // top of the panel); the factor is applied to all rows
  dion_ctx* c = s.c;
  const bool adaptive = (mode == RM_ADAPTIVE);
  const bool skips = rm_skips(mode);
  const int* skip = skips ? (s.os + OS_DONE) : nullptr;
  if (mode == RM_CHECKED) {
    // CholeskyQR2, second round: first measure the first round's result; orthonormal enough -> done, and
    // everything below is skipped on the device
    DION_TRY(probe(s, pin_off, rows, r, probe_phase));
  }
  GemmArgs g = gemm_args();
  g.M = r; g.N = r; g.K = gram_rows > 0 ? gram_rows : rows;
  g.A = s.ws + pin_off; g.a_si = 1; g.a_sk = r;
  g.B = s.ws + pin_off; g.b_sk = r; g.b_sn = 1;
  if (gram_rows == 0 && gram_on_pairs(s, rows, r)) {
    // The Gram matrix of a tall panel on half pairs: the panel is scaled and split into Pout's buffer (free until
    // the solve writes it) and the product takes three kind::f16 MMAs per K step instead of the three or four
    // kind::tf32 ones; the same 22 significant bits.  1 / scale^2 reaches the epilogue through a device scalar.
    const int* sk = skips ? skip : nullptr;
    __half* hi = reinterpret_cast<__half*>(s.ws + pout_off);
    __half* lo = hi + rows * r;
    i64 parts = (rows * r / 4 + 2047) / 2048;
    if (parts > AMAX_PARTS) parts = AMAX_PARTS;
    launch_pdl(k_absmax_partial, dim3((unsigned)parts, (unsigned)s.nb), dim3(256), 0, s.st, (const float*)(s.ws + pin_off), r, rows, r,
               s.ws + s.L.gmax, s.wstride, sk, (i64)OS_SLOT_INTS);
    DION_CHECK_LAUNCH(c);
    launch_pdl(k_split_f16_scaled, dim3((unsigned)grid_for(c, rows * r / 8), (unsigned)s.nb), dim3(256), 0, s.st,
               (const float*)(s.ws + pin_off), r, rows, r, (const float*)(s.ws + s.L.gmax), (int)parts, hi, lo, s.ws + s.L.gmax + AMAX_PARTS,
               s.wstride, sk, (i64)OS_SLOT_INTS, -1.f, (const float*)nullptr);
    DION_CHECK_LAUNCH(c);
    g.ab16 = 1; g.f16 = 1;
    g.A = reinterpret_cast<const float*>(hi); g.A16lo = lo;
    g.B = reinterpret_cast<const float*>(hi); g.B16lo = lo;
    g.alpha_dev = s.ws + s.L.gmax + AMAX_PARTS; g.alpha_dev_stride = s.wstride;
  }
  g.C = s.ws + s.L.Gram; g.ldc = r; g.epi = EPI_STORE; g.tri = TRI_LOWER; g.skip_flag = skips ? skip : nullptr; g.precise = rm_precise(mode) ? 1 : 0;
  DION_TRY(launch_gemm_chain(s, g));
  launch_pdl(k_round_begin, dim3((unsigned)(s.nb)), dim3(256), 0, s.st, s.ws + s.L.Gram, r, r, 0.f, s.ws + s.L.gdiag, s.ws + s.L.scal, s.os,
                                        skips ? 1 : 0, s.wstride, c->dev_ints);
  DION_CHECK_LAUNCH(c);
  // Tall panels with r > 512: blocked triangular solve with the 512-column diagonal inverses
  // only (the levels of the triangular inverse above 512 are never formed).
  // alone, 512-column products need >= 128 row tiles to fill the GPU; beside the factorization
  // (second stream) they are background work at any height
  const bool trsm = (r > NBO) && (rows >= 8192 || c->side != nullptr);
  if (skips && passthrough) {   // a finished panel is passed through (before anything writes Pout)
    dim3 grid((unsigned)grid_for(c, rows * r), (unsigned)s.nb);
    launch_pdl(k_copy_panel, grid, dim3(256), 0, s.st, s.ws + pin_off, r, s.ws + pout_off, r, rows, r, nullptr, s.os + OS_DONE, s.wstride);
    DION_CHECK_LAUNCH(c);
  }
  if (trsm) {
    // Pout_J = (Pin_J - sum_{K<J} Pout_K L_{J,K}^T) Linv_JJ^T, block columns J of 512.
    // The solves run with the plain 3xTF32 product: their rounding error enters U once (~1e-6),
    // whereas an error in the Gram matrix or its factor is amplified by the panel's conditioning.
    // Block column J needs row block J of the factor and the inverse of its diagonal square, both
    // final once the factorization has passed J: the solves run on a second stream beside the rest
    // of the factorization, whose serial 64-column chain leaves most SMs idle.
    const float* Lm = s.ws + s.L.Gram;     // the factor, lower
    float* Wt = s.ws + (s.wt_off >= 0 ? s.wt_off : s.L.R);   // rows x 512 temporary (R is free during the orthonormalization)
    // On tall panels the two products of a block column run on scaled half pairs (22 significant bits in three
    // kind::f16 MMAs; 1024-k chains) like the Gram matrix: the right-hand side, the factor's row block and the
    // diagonal inverse are scaled by powers of two found on the device, the finished columns of Pout (entries of
    // an orthonormal basis; at most 1 / sqrt(pivot floor) = 100 in a deflating round) by 2^6.
    const bool spairs = s.wt_off < 0 && s.L.SolveP > 0 && solve_on_pairs(s, rows, r, mode);
    auto absmax_split = [&](const float* src, i64 ld, i64 nrows, i64 ncols, i64 out_off, i64 slot, float other_inv,
                            const float* other_dev) -> int {
      // pair of the nrows x ncols block at `src` (slice-relative pointer of matrix 0) into scratch at out_off; the
      // scale factor goes to smax slot `slot`
      i64 parts = (nrows * ncols / 4 + 2047) / 2048;
      if (parts < 1) parts = 1;
      if (parts > AMAX_PARTS) parts = AMAX_PARTS;
      float* pm = s.ws + s.L.smax + slot * (AMAX_PARTS + 64);
      launch_pdl(k_absmax_partial, dim3((unsigned)parts, (unsigned)s.nb), dim3(256), 0, s.st, src, ld, nrows, ncols, pm, s.wstride, skip,
                 (i64)OS_SLOT_INTS);
      DION_CHECK_LAUNCH(c);
      __half* hi = reinterpret_cast<__half*>(s.ws + out_off);
      launch_pdl(k_split_f16_scaled, dim3((unsigned)grid_for(c, nrows * ncols / 8), (unsigned)s.nb), dim3(256), 0, s.st, src, ld, nrows, ncols,
                 (const float*)pm, (int)parts, hi, hi + nrows * ncols, pm + AMAX_PARTS, s.wstride, skip, (i64)OS_SLOT_INTS, other_inv, other_dev);
      DION_CHECK_LAUNCH(c);
      return DION_OK;
    };
    auto solve_block_pairs = [&](i64 J0, i64 sz) -> int {
      const float* rhs = s.ws + pin_off + J0;
      i64 rhs_ld = r;
      __half* pop = reinterpret_cast<__half*>(s.ws + s.L.S16);          // pair of Pout: rows x r, dense
      const float* sc = s.ws + s.L.smax;
      if (J0 > 0) {
        // W = rhs - Pout[:, :J0] L[J0:J0+sz, :J0]^T
        DION_TRY(absmax_split(Lm + J0 * r, r, sz, J0, s.L.LfP, 0, ldexpf(1.f, -6), nullptr));
        __half* lh = reinterpret_cast<__half*>(s.ws + s.L.LfP);
        GemmArgs w = gemm_args();
        w.M = rows; w.N = sz; w.K = J0;
        w.ab16 = 1; w.f16 = 1;
        w.A = (const float*)pop; w.A16lo = pop + rows * r; w.a_si = r; w.a_sk = 1;
        w.B = (const float*)lh; w.B16lo = lh + sz * J0; w.b_sk = 1; w.b_sn = J0;
        w.C = Wt; w.ldc = NBO; w.epi = EPI_C2_SUB; w.C2 = rhs; w.ldc2 = r; w.c2_mode = ADD_F32;
        w.alpha_dev = sc + AMAX_PARTS; w.alpha_dev_stride = s.wstride;
        w.skip_flag = skip;
        DION_TRY(launch_gemm_chain(s, w, true));
        rhs = Wt; rhs_ld = NBO;
      }
      // V = rhs Linv_JJ^T
      DION_TRY(absmax_split(rhs, rhs_ld, rows, sz, s.L.SolveP, 1, 1.f, nullptr));
      const i64 li_off = s.L.LfP + NBO * r;
      DION_TRY(absmax_split(s.ws + s.L.Linv + J0 * r + J0, r, sz, sz, li_off, 2, 1.f, sc + (AMAX_PARTS + 64) + AMAX_PARTS));
      __half* rh = reinterpret_cast<__half*>(s.ws + s.L.SolveP);
      __half* ih = reinterpret_cast<__half*>(s.ws + li_off);
      GemmArgs v = gemm_args();
      v.M = rows; v.N = sz; v.K = sz;
      v.ab16 = 1; v.f16 = 1;
      v.A = (const float*)rh; v.A16lo = rh + rows * sz; v.a_si = sz; v.a_sk = 1;
      v.B = (const float*)ih; v.B16lo = ih + sz * sz; v.b_sk = 1; v.b_sn = sz; v.klimit = 1;
      v.C = s.ws + pout_off + J0; v.ldc = r; v.epi = EPI_STORE; v.skip_flag = skip;
      v.alpha_dev = sc + 2 * (AMAX_PARTS + 64) + AMAX_PARTS; v.alpha_dev_stride = s.wstride;
      DION_TRY(launch_gemm_chain(s, v));
      if (J0 + sz < r) {      // the new block column of Pout joins the pair (later block columns read it)
        ChainPtrs t;
        for (int b = 0; b < s.nb; ++b) t.p[b] = s.W(b, pout_off + J0);
        launch_pdl(k_split_f16_fixed, dim3((unsigned)grid_for(c, rows * sz / 8), (unsigned)s.nb), dim3(256), 0, s.st, t, r, rows, sz,
                   ldexpf(1.f, 6), pop + J0, pop + rows * r + J0, s.wstride, r, skip, (i64)OS_SLOT_INTS);
        DION_CHECK_LAUNCH(c);
      }
      return DION_OK;
    };
    auto solve_block = [&](i64 J0, i64 sz) -> int {
      if (spairs && sz >= 64 && sz % 8 == 0) return solve_block_pairs(J0, sz);
      const float* rhs = s.ws + pin_off + J0;
      i64 rhs_ld = r;
      if (J0 > 0) {
        GemmArgs w = gemm_args();
        w.M = rows; w.N = sz; w.K = J0;
        w.A = s.ws + pout_off; w.a_si = r; w.a_sk = 1;
        w.B = Lm + J0 * r; w.b_sk = 1; w.b_sn = r;
        w.C = Wt; w.ldc = NBO; w.epi = EPI_C2_SUB; w.C2 = rhs; w.ldc2 = r; w.c2_mode = ADD_F32;
        w.skip_flag = skip;
        DION_TRY(launch_gemm_chain(s, w, true));
        rhs = Wt; rhs_ld = NBO;
      }
      GemmArgs v = gemm_args();
      v.M = rows; v.N = sz; v.K = sz;
      v.A = rhs; v.a_si = rhs_ld; v.a_sk = 1;
      v.B = s.ws + s.L.Linv + J0 * r + J0; v.b_sk = 1; v.b_sn = r; v.klimit = 1;
      v.C = s.ws + pout_off + J0; v.ldc = r; v.epi = EPI_STORE; v.skip_flag = skip;
      DION_TRY(launch_gemm_chain(s, v));
      return DION_OK;
    };
    if (c->side != nullptr) {
      cudaStream_t main_st = s.st;
      auto next_event = [&]() { cudaEvent_t e = c->side_ev[c->side_cursor]; c->side_cursor = (c->side_cursor + 1) % 32; return e; };
      const std::function<int(i64, i64)> after_block = [&](i64 J0, i64 sz) -> int {
        cudaEvent_t e = next_event();
        if (cudaEventRecord(e, main_st) != cudaSuccess || cudaStreamWaitEvent(c->side, e, 0) != cudaSuccess) return DION_ERR_CUDA;
        s.st = c->side; s.no_split = true;
        const int rc = solve_block(J0, sz);
        s.st = main_st; s.no_split = false;
        return rc;
      };
      DION_TRY(potrf_trtri(s, r, mode, false, &after_block));
      cudaEvent_t e = next_event();   // join: the round ends when the last solve has finished
      if (cudaEventRecord(e, c->side) != cudaSuccess || cudaStreamWaitEvent(main_st, e, 0) != cudaSuccess) return DION_ERR_CUDA;
    } else {
      DION_TRY(potrf_trtri(s, r, mode, false));
      for (i64 J0 = 0; J0 < r; J0 += NBO) DION_TRY(solve_block(J0, (r - J0 < NBO) ? (r - J0) : NBO));
    }
    if (adaptive) {
      launch_pdl(k_round_end, dim3((unsigned)(s.nb)), dim3(1), 0, s.st, s.os, GOOD_REL, DONE_REL, c->dev_ints + 2);
      DION_CHECK_LAUNCH(c);
    }
    return DION_OK;
  }
  DION_TRY(potrf_trtri(s, r, mode, true));
  GemmArgs u = gemm_args();
  u.M = rows; u.N = r; u.K = r;
  u.A = s.ws + pin_off; u.a_si = r; u.a_sk = 1;
  u.B = s.ws + s.L.Linv; u.b_sk = 1; u.b_sn = r; u.klimit = 1;
  u.C = s.ws + pout_off; u.ldc = r; u.epi = EPI_STORE; u.skip_flag = skip;
  DION_TRY(launch_gemm_chain(s, u));
  if (adaptive) {
    launch_pdl(k_round_end, dim3((unsigned)(s.nb)), dim3(1), 0, s.st, s.os, GOOD_REL, DONE_REL, c->dev_ints + 2);
    DION_CHECK_LAUNCH(c);
  }
  return DION_OK;
}

// Householder factorization of the rows x r matrix A (ld = r): reflectors into V, the triangular
// factor into the rows of A above the diagonal and its diagonal into the matrix's d scratch.
int householder_factor(StepCtx& s, float* A, float* V, i64 rows, i64 r, int b) {
  dion_ctx* c = s.c;
  float* diag = s.W(b, s.L.d);
  for (i64 j = 0; j < r; ++j) {
    k_hh_reflector<<<1, 1024, 0, s.st>>>(A, r, rows, j, V, r, diag);
    DION_CHECK_LAUNCH(c);
    if (j + 1 < r) {
      const unsigned gx = (unsigned)((r - j - 1 + 31) / 32);
      k_hh_apply<<<gx, 256, 0, s.st>>>(A, r, rows, j, V, r, j, j + 1, r);
      DION_CHECK_LAUNCH(c);
    }
  }
  return DION_OK;
}

int householder(StepCtx& s, float* A, float* V, i64 rows, i64 r, int b) {
  dion_ctx* c = s.c;
  float* diag = s.W(b, s.L.d);
  DION_TRY(householder_factor(s, A, V, rows, r, b));
  {
    const i64 total = rows * r;
    int blocks = (int)((total + 255) / 256);
    if (blocks > 8 * c->sm_count) blocks = 8 * c->sm_count;
    k_set_identity<<<blocks, 256, 0, s.st>>>(A, r, rows, r);
    DION_CHECK_LAUNCH(c);
    for (i64 j = r - 1; j >= 0; --j) {
      // columns < j of the partial product are still unit vectors e_c with c < j: untouched
      const unsigned gx = (unsigned)((r - j + 31) / 32);
      k_hh_apply<<<gx, 256, 0, s.st>>>(A, r, rows, j, V, r, j, j, r);
      DION_CHECK_LAUNCH(c);
    }
    k_sign_fix<<<blocks, 256, 0, s.st>>>(A, r, rows, r, diag);
    DION_CHECK_LAUNCH(c);
  }
  return DION_OK;
}

// Adaptive rounds on the panel at off_a (ping-pong with off_b; the result ends at off_a): the device
// decides after each round whether the panel is done.
int adaptive_rounds(StepCtx& s, i64 off_a, i64 off_b, i64 rows, i64 r, i64 gram_rows) {
  static_assert(MAX_ROUNDS % 2 == 0, "the result must end in the first buffer");
  for (int it = 0; it < MAX_ROUNDS; it += 2) {
    DION_TRY(cholqr_round(s, off_a, off_b, rows, r, RM_ADAPTIVE, gram_rows));
    DION_TRY(cholqr_round(s, off_b, off_a, rows, r, RM_ADAPTIVE, gram_rows));
  }
  launch_pdl(k_orth_finish, dim3((unsigned)(s.nb)), dim3(1), 0, s.st, s.os, s.c->dev_ints);
  s.c->launches++;
  if (cudaGetLastError() != cudaSuccess) return DION_ERR_CUDA;
  return DION_OK;
}

// Randomized Cholesky QR (Algorithm 4 on one device) of the rows x r panel in P0 of every
// matrix of the chain; U ends in P0.
//   Pt = S P (k x r sketch).  R1 = triangular factor of QR(Pt): computed by deflating Cholesky-QR
//   rounds on the sketch, never formed explicitly -- the rounds run on the stacked panel [Pt; P] with
//   their Gram matrices taken from the sketch rows only, so every round's triangular factor is applied
//   to the sketch and to P at once; when the sketch has become orthonormal, the lower rows hold
//   B = P R1^-1.  Then Cholesky QR on B (R2 = Cholesky(B^T B), U = B R2^-1; a second pass only if the
//   device's check asks for it).  All matrices of a chain have the same number of sketch rows.
int rcqr(StepCtx& s, i64 rows, i64 r) {
  dion_ctx* c = s.c;
  if (s.list == nullptr) return DION_ERR_INVALID;
  const i64 k = s.list[0]->sketch_rows;
  for (int b = 0; b < s.nb; ++b) {
    const dion_matrix* a = s.list[b];
    if (a->sketch_rows != k) return DION_ERR_INVALID;
    float* stack = s.W(b, s.L.Sk);
    GemmArgs g = gemm_args();
    g.M = k; g.N = r; g.K = rows;
    g.A = (const float*)a->sketch; g.a_si = a->ld_sketch; g.a_sk = 1;
    g.B = s.W(b, s.L.P0); g.b_sk = r; g.b_sn = 1;
    g.C = stack; g.ldc = r; g.epi = EPI_STORE; g.precise = 1;
    DION_TRY(launch_gemm(s, g, b));
    dim3 grid((unsigned)grid_for(c, rows * r), 1);
    launch_pdl(k_copy_block, grid, dim3(256), 0, s.st, (const float*)s.W(b, s.L.P0), r, stack + k * r, r, rows, r, nullptr, 0);
    DION_CHECK_LAUNCH(c);
  }
  s.wt_off = s.L.SkW;
  const int rc = adaptive_rounds(s, s.L.Sk, s.L.SkV, k + rows, r, k);
  s.wt_off = -1;
  DION_TRY(rc);
  // B = the panel rows of the stack; the step's state slot starts afresh for its Cholesky QR
  launch_pdl(k_reset_rounds, dim3((unsigned)s.nb), dim3(1), 0, s.st, s.os);
  DION_CHECK_LAUNCH(c);
  DION_TRY(cholqr_round(s, s.L.Sk + k * r, s.L.P1, rows, r, RM_FIRST));
  return cholqr_round(s, s.L.P1, s.L.P0, rows, r, RM_CHECKED);
}

// The orthonormalization a step on (m, n, r) will use.
int resolve_orth(const dion_ctx* c, i64 r, i64 short_dim) {
  int mode = c->cfg.orth;
  if (mode == DION_ORTH_AUTO) mode = (4 * r <= short_dim) ? DION_ORTH_CHOLQR2 : DION_ORTH_SHIFTED3;
  return mode;
}

// ... for a chain with (step) or without (Lazy-Dion, data-parallel calls) the sketches of the RCQR mode.
int resolve_orth_for(const dion_ctx* c, i64 r, i64 short_dim, bool has_sketches) {
  int mode = resolve_orth(c, r, short_dim);
  if (mode == DION_ORTH_RCQR && !has_sketches) mode = (4 * r <= short_dim) ? DION_ORTH_CHOLQR2 : DION_ORTH_SHIFTED3;
  return mode;
}

// Where the product that forms the panel writes it: CholeskyQR2 reads it from the save buffer (round one goes
// Psave -> P1, round two P1 -> P0), so that the panel is still there if a pivot fails; every other mode works in P0.
i64 panel_offset(const StepCtx& s, i64 r, i64 short_dim) {
  const bool cq2 = resolve_orth_for(s.c, r, short_dim, s.list != nullptr) == DION_ORTH_CHOLQR2;
  return (cq2 && s.L.Psave > 0) ? s.L.Psave : s.L.P0;
}

// The device-side fallback of CholeskyQR2 (k_cgs_fallback): one cooperative launch over the chain's matrices.
int cgs_fallback(StepCtx& s, i64 pin_off, i64 pout_off, i64 rows, i64 r) {
  dion_ctx* c = s.c;
  i64 G = rows / 8;
  if (G < 1) G = 1;
  if (G > c->sm_count) G = c->sm_count;
  const float* Pin = s.ws + pin_off;
  float* U = s.ws + pout_off;
  float* part = s.ws + s.L.fb_part;
  float* hvec = s.ws + s.L.fb_h;
  float* npart = s.ws + s.L.fb_n;
  int* os = s.os;
  int* status = c->dev_ints;
  int* fallbacks = c->dev_ints + 3;
  i64 ld = r, wstride = s.wstride;
  int nb = s.nb;
  long long limit = umma::SPIN_LIMIT_CYCLES;
  void* args[] = {&Pin, &U, &ld, &rows, &r, &part, &hvec, &npart, &os, &status, &fallbacks, &wstride, &nb, &limit};
  if (cudaLaunchCooperativeKernel((const void*)k_cgs_fallback, dim3((unsigned)G), dim3(256), args, 0, s.st) != cudaSuccess) {
    cudaGetLastError();
    return DION_ERR_CUDA;
  }
  c->launches++;
  return DION_OK;
}

bool fallback_fits(const dion_ctx* c, i64 rows) {
  return (rows + c->sm_count - 1) / c->sm_count <= CGS_MAX_ROWS_PER_CTA;
}

// Orthonormalize the rows x r panel at pin_off (= panel_offset) of every matrix of the chain; *U_off is the
// scratch offset of the buffer that holds U afterwards.
int orthonormalize(StepCtx& s, i64 rows, i64 r, i64 short_dim, i64 pin_off, i64* U_off) {
  const int mode = resolve_orth_for(s.c, r, short_dim, s.list != nullptr);
  if (mode == DION_ORTH_CHOLQR2) {
    // the first round with the accurate products; the second one only if the first one's result is
    // not yet orthonormal to ORTH_TAU_F (measured by the probe).  A pivot that is not positive in
    // either round (the paper's "CQR failure") raises the step's fail flag only; the fallback kernel then
    // orthonormalizes the saved panel and clears the flag, or confirms the breakdown.
    const bool fb = pin_off != s.L.P0 && fallback_fits(s.c, rows);
    if (r <= NB && rows <= TINY_MAX_ROWS && s.redo_p == nullptr) {
      // a panel that fits one CTA's shared memory: both rounds and the test between them in one launch
      launch_pdl(k_tiny_cholqr2, dim3((unsigned)s.nb), dim3(TINY_THREADS), (size_t)tiny_cholqr2_smem(rows), s.st, (const float*)(s.ws + pin_off),
                 s.ws + s.L.P0, (int)rows, (int)r, s.os, ORTH_TAU_F, s.c->dev_ints + 2, fb ? (int*)nullptr : s.c->dev_ints, s.c->dev_ints,
                 s.wstride);
      DION_CHECK_LAUNCH(s.c);
      if (fb) DION_TRY(cgs_fallback(s, pin_off, s.L.P0, rows, r));
      *U_off = s.L.P0;
      return DION_OK;
    }
    s.quiet_fail = fb;
    // Round one writes P0, where U is expected; the second round, when it runs, goes P0 -> P1 and is copied
    // back: the common case (one round) moves the panel once.
    int rc = cholqr_round(s, pin_off, s.L.P0, rows, r, RM_FIRST);
    const bool redo = s.redo_p != nullptr;
    if (redo) {
      // The panel came from the fast product (bf16 operand pairs, ~1e-5): good enough exactly when the panel is well
      // conditioned, which the probe of the first round's result shows.  Otherwise the device recomputes the panel
      // with the accurate product and repeats the round; all of that is launched and skipped in the common case.
      if (rc == DION_OK) rc = probe(s, s.L.P0, rows, r, PROBE_FAST);
      if (rc == DION_OK) rc = (*s.redo_p)();
      if (rc == DION_OK) rc = cholqr_round(s, pin_off, s.L.P0, rows, r, RM_REDO, 0, false);
    }
    if (rc == DION_OK) rc = cholqr_round(s, s.L.P0, s.L.P1, rows, r, RM_CHECKED, 0, false, redo ? PROBE_AFTER_REDO : PROBE_CHECK);
    s.quiet_fail = false;
    DION_TRY(rc);
    {
      dim3 grid((unsigned)grid_for(s.c, rows * r), (unsigned)s.nb);
      launch_pdl(k_copy_panel, grid, dim3(256), 0, s.st, (const float*)(s.ws + s.L.P1), r, s.ws + s.L.P0, r, rows, r,
                 (const int*)(s.os + OS_DONE), (const int*)nullptr, s.wstride);
      DION_CHECK_LAUNCH(s.c);
    }
    if (fb) DION_TRY(cgs_fallback(s, pin_off, s.L.P0, rows, r));   // else: the failed pivot was reported as a breakdown
    *U_off = s.L.P0;
  } else if (mode == DION_ORTH_SHIFTED3) {
    DION_TRY(adaptive_rounds(s, s.L.P0, s.L.P1, rows, r, 0));
    *U_off = s.L.P0;
  } else if (mode == DION_ORTH_RCQR) {
    DION_TRY(rcqr(s, rows, r));
    *U_off = s.L.P0;
  } else {
    for (int m = 0; m < s.nb; ++m) DION_TRY(householder(s, s.W(m, s.L.P0), s.W(m, s.L.P1), rows, r, m));
    *U_off = s.L.P0;
  }
  return DION_OK;
}

// ColNorm of matrix b's W (rows x r, ld = r) into `out`.
int colnorm(StepCtx& s, int b, const float* W, i64 rows, i64 r, float* out, i64 ldo, float* d_out,
            const int* skip = nullptr, i64 ldw = 0) {
  if (ldw == 0) ldw = r;
  dion_ctx* c = s.c;
  int chunks; i64 per;
  colnorm_plan(rows, r, c->sm_count, &chunks, &per);
  float* part = s.W(b, s.L.cn_part);
  dim3 grid((unsigned)((r + 127) / 128), (unsigned)chunks);
  launch_pdl(k_colsumsq_partial, grid, dim3(128), 0, s.st, W, ldw, rows, r, per, part, (const int*)nullptr, (i64)0);
  DION_CHECK_LAUNCH(c);
  launch_pdl(k_colnorm_apply, grid, dim3(128), 0, s.st, W, ldw, rows, r, per, chunks, (const float*)part, c->cfg.eps, out, ldo,
             s.W(b, s.L.d), d_out, c->dev_ints, skip != nullptr ? skip : (const int*)(s.OS(b) + OS_FAIL), (i64)0, ChainPtrs(), ChainPtrs());
  DION_CHECK_LAUNCH(c);
  return DION_OK;
}

// ---- elementwise kernels over a whole chain -------------------------------------------------------------------
// Each helper makes ONE launch over the chain's matrices (blockIdx.y or .z) when their arrays share leading
// dimensions and alignment, else one launch per matrix; outputs are in the scratch slices either way.

// ColNorm of every matrix's R (scratch, rows x r dense) into its Q, d exported to colnorm_out.
int colnorm_chain(StepCtx& s, const dion_matrix* const* list, i64 rows, i64 r) {
  dion_ctx* c = s.c;
  bool one = s.nb > 1 && s.nb <= GEMM_TAB_MAX && c->chain_batch;
  for (int b = 1; b < s.nb && one; ++b) one = list[b]->ldq == list[0]->ldq;
  if (!one) {
    for (int b = 0; b < s.nb; ++b)
      DION_TRY(colnorm(s, b, s.W(b, s.L.R), rows, r, (float*)list[b]->Q, list[b]->ldq, list[b]->colnorm_out));
    return DION_OK;
  }
  int chunks; i64 per;
  colnorm_plan(rows, r, c->sm_count, &chunks, &per);
  ChainPtrs Qs, ds;
  for (int b = 0; b < s.nb; ++b) { Qs.p[b] = list[b]->Q; ds.p[b] = list[b]->colnorm_out; }
  dim3 grid((unsigned)((r + 127) / 128), (unsigned)chunks, (unsigned)s.nb);
  launch_pdl(k_colsumsq_partial, grid, dim3(128), 0, s.st, (const float*)(s.ws + s.L.R), r, rows, r, per, s.ws + s.L.cn_part,
             (const int*)nullptr, s.wstride);
  DION_CHECK_LAUNCH(c);
  launch_pdl(k_colnorm_apply, grid, dim3(128), 0, s.st, (const float*)(s.ws + s.L.R), r, rows, r, per, chunks,
             (const float*)(s.ws + s.L.cn_part), c->cfg.eps, (float*)nullptr, list[0]->ldq, s.ws + s.L.d, (float*)nullptr, c->dev_ints,
             (const int*)(s.os + OS_FAIL), s.wstride, Qs, ds);
  DION_CHECK_LAUNCH(c);
  return DION_OK;
}

// hi / lo bf16 pair of src[b] (rows x cols, leading dimension ld[b]) into the scratch slices at out_off.
// skip0: the flag of matrix 0 (a state slot apart per matrix), or nullptr.
// copy_off >= 0 (chain launch only): a dense fp32 copy of the sources in the scratch slices too; *copied says whether it was made.
int split_chain(StepCtx& s, const float* const* src, const i64* ld, i64 rows, i64 cols, i64 out_off, const int* skip0,
                i64 copy_off = -1, bool* copied = nullptr) {
  dion_ctx* c = s.c;
  bool one = s.nb > 1 && s.nb <= GEMM_TAB_MAX && c->chain_batch;
  for (int b = 1; b < s.nb && one; ++b) one = ld[b] == ld[0];
  const unsigned gx = (unsigned)grid_for(c, rows * cols / 8);
  if (one) {
    ChainPtrs t;
    for (int b = 0; b < s.nb; ++b) t.p[b] = src[b];
    __nv_bfloat16* hi = reinterpret_cast<__nv_bfloat16*>(s.ws + out_off);
    launch_pdl(k_split_bf16_chain, dim3(gx, (unsigned)s.nb), dim3(256), 0, s.st, t, ld[0], rows, cols, hi, hi + rows * cols, s.wstride, skip0,
               (i64)OS_SLOT_INTS, copy_off >= 0 ? s.ws + copy_off : (float*)nullptr);
    DION_CHECK_LAUNCH(c);
    if (copied != nullptr) *copied = copy_off >= 0;
    return DION_OK;
  }
  if (copied != nullptr) *copied = false;
  for (int b = 0; b < s.nb; ++b) {
    __nv_bfloat16* hi = reinterpret_cast<__nv_bfloat16*>(s.W(b, out_off));
    launch_pdl(k_split_bf16, dim3(gx), dim3(256), 0, s.st, src[b], ld[b], rows, cols, hi, hi + rows * cols,
               skip0 != nullptr ? skip0 + (i64)b * OS_SLOT_INTS : (const int*)nullptr);
    DION_CHECK_LAUNCH(c);
  }
  return DION_OK;
}

// src[b] rounded to TF32 into the scratch slices at out_off.
// half_scale > 0: IEEE half values of half_scale * src instead (see x_half).
int round_chain(StepCtx& s, const float* const* src, const i64* ld, i64 rows, i64 cols, i64 out_off, const int* skip0,
                float half_scale = 0.f) {
  dion_ctx* c = s.c;
  bool one = s.nb > 1 && s.nb <= GEMM_TAB_MAX && c->chain_batch;
  for (int b = 1; b < s.nb && one; ++b) one = ld[b] == ld[0];
  if (half_scale > 0.f) {
    const unsigned g8 = (unsigned)grid_for(c, rows * cols / 8);
    if (one) {
      ChainPtrs t;
      for (int b = 0; b < s.nb; ++b) t.p[b] = src[b];
      launch_pdl(k_round_f16_chain, dim3(g8, (unsigned)s.nb), dim3(256), 0, s.st, t, ld[0], rows, cols, half_scale,
                 reinterpret_cast<__half*>(s.ws + out_off), s.wstride, skip0, (i64)OS_SLOT_INTS);
      DION_CHECK_LAUNCH(c);
      return DION_OK;
    }
    for (int b = 0; b < s.nb; ++b) {
      launch_pdl(k_round_f16, dim3(g8), dim3(256), 0, s.st, src[b], ld[b], rows, cols, half_scale, reinterpret_cast<__half*>(s.W(b, out_off)),
                 skip0 != nullptr ? skip0 + (i64)b * OS_SLOT_INTS : (const int*)nullptr);
      DION_CHECK_LAUNCH(c);
    }
    return DION_OK;
  }
  const unsigned gx = (unsigned)grid_for(c, rows * cols / 4);
  if (one) {
    ChainPtrs t;
    for (int b = 0; b < s.nb; ++b) t.p[b] = src[b];
    launch_pdl(k_round_tf32_chain, dim3(gx, (unsigned)s.nb), dim3(256), 0, s.st, t, ld[0], rows, cols, s.ws + out_off, s.wstride, skip0,
               (i64)OS_SLOT_INTS);
    DION_CHECK_LAUNCH(c);
    return DION_OK;
  }
  for (int b = 0; b < s.nb; ++b) {
    launch_pdl(k_round_tf32, dim3(gx), dim3(256), 0, s.st, src[b], ld[b], rows, cols, s.W(b, out_off),
               skip0 != nullptr ? skip0 + (i64)b * OS_SLOT_INTS : (const int*)nullptr);
    DION_CHECK_LAUNCH(c);
  }
  return DION_OK;
}

bool overlap(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
  return a0 < b0 + nb && b0 < a0 + na;
}

// shard: `a` describes a column shard of a wider matrix (the sharded calls): r may exceed its n.
int validate(const dion_matrix* a, bool shard = false) {
  if (a == nullptr) return DION_ERR_INVALID;
  if (a->X == nullptr || a->M == nullptr || a->G == nullptr || a->Q == nullptr) return DION_ERR_INVALID;
  if (a->g_dtype != DION_F32 && a->g_dtype != DION_BF16) return DION_ERR_INVALID;
  if (a->m < 1 || a->n < 1) return DION_ERR_SHAPE;
  if (a->r < 1 || a->r > a->m || (!shard && a->r > a->n)) return DION_ERR_SHAPE;
  if (a->ldx < a->n || a->ldm < a->n || a->ldg < a->n || a->ldq < a->r) return DION_ERR_SHAPE;
  if (a->transposed != 0 && a->transposed != 1) return DION_ERR_INVALID;
  const i64 qrows = a->transposed ? a->m : a->n;
  const size_t gsz = (a->g_dtype == DION_BF16) ? 2 : 4;
  if (((uintptr_t)a->X & 3) || ((uintptr_t)a->M & 3) || ((uintptr_t)a->Q & 3) || ((uintptr_t)a->G & (gsz - 1)))
    return DION_ERR_ALIGN;
  if (a->colnorm_out != nullptr && ((uintptr_t)a->colnorm_out & 3)) return DION_ERR_ALIGN;
  const size_t nx = (size_t)((a->m - 1) * a->ldx + a->n) * 4, nm = (size_t)((a->m - 1) * a->ldm + a->n) * 4;
  const size_t ng = (size_t)((a->m - 1) * a->ldg + a->n) * gsz, nq = (size_t)((qrows - 1) * a->ldq + a->r) * 4;
  if (overlap(a->X, nx, a->M, nm) || overlap(a->X, nx, a->G, ng) || overlap(a->X, nx, a->Q, nq) ||
      overlap(a->M, nm, a->G, ng) || overlap(a->M, nm, a->Q, nq) || overlap(a->G, ng, a->Q, nq))
    return DION_ERR_ALIAS;
  if (a->colnorm_out != nullptr) {
    const size_t nc = (size_t)a->r * 4;
    if (overlap(a->colnorm_out, nc, a->X, nx) || overlap(a->colnorm_out, nc, a->M, nm) ||
        overlap(a->colnorm_out, nc, a->G, ng) || overlap(a->colnorm_out, nc, a->Q, nq))
      return DION_ERR_ALIAS;
  }
  return DION_OK;
}

int begin_step(dion_ctx* c, const dion_matrix* a, int nb, cudaStream_t st, StepCtx* s, int fixed_slot = -1) {
  s->c = c;
  s->st = st;
  s->L = make_layout(c, a->m, a->n, a->r);
  s->ws = c->ws;
  s->nb = nb;
  s->wstride = s->L.total;
  if (fixed_slot >= 0) {
    s->os = c->dev_ints + 8 + (i64)fixed_slot * OS_SLOT_INTS;
  } else {
    if (c->flag_cursor + nb > MAX_FLAG_SLOTS - MAX_GRAPHS) c->flag_cursor = 0;   // the slots of a chain are contiguous
    s->os = c->dev_ints + 8 + (i64)c->flag_cursor * OS_SLOT_INTS;
    c->flag_cursor = (c->flag_cursor + nb) % (MAX_FLAG_SLOTS - MAX_GRAPHS);
  }
  s->flag = s->os + OS_FAIL;
  s->tensor = (c->cfg.engine != DION_ENGINE_SIMT);
  s->in_orth = false;
  if (cudaMemsetAsync(s->os, 0, sizeof(int) * OS_SLOT_INTS * nb, st) != cudaSuccess) return DION_ERR_CUDA;
  return DION_OK;
}

// R = (M + G)^T U on bf16 pairs (transposed form: (M + G) U): where M + G is kept in scratch (sum_in_scratch) the
// product runs on the bf16 (hi, lo) pair of the sum and of U, three bf16 MMAs per K step (1.3 TF32 passes instead of
// three); it is accurate to ~1e-5, which is what Q <- ColNorm(R) and the error feedback need of it.
bool r_on_pairs(const StepCtx& s, i64 m, i64 n, i64 r) {
  return s.tensor && s.c->cfg.precision == DION_PREC_FP32 && s.L.B32 > 0 && s.L.Bp > 0 && m >= 128 && n >= 128 && r >= 64;
}

// Forms M + G in scratch (fp32) and, when `pair`, as a bf16 pair beside it.
int form_sum(StepCtx& s, int b, const dion_matrix* a, bool pair) {
  dion_ctx* c = s.c;
  const i64 m = a->m, n = a->n;
  const bool vec = !((uintptr_t)a->M & 15) && a->ldm % 4 == 0 &&
                   (a->g_dtype == DION_BF16 ? (!((uintptr_t)a->G & 7) && a->ldg % 4 == 0)
                                            : (!((uintptr_t)a->G & 15) && a->ldg % 4 == 0));
  const int g_mode = (a->g_dtype == DION_BF16) ? ADD_BF16 : ADD_F32;
  const int grid = grid_for(c, m * n / 4);
  __nv_bfloat16* bh = pair ? reinterpret_cast<__nv_bfloat16*>(s.W(b, s.L.Bp)) : nullptr;
  __nv_bfloat16* bl = pair ? bh + m * n : nullptr;
  if (vec) launch_pdl(k_form_b32<true>, grid, dim3(256), 0, s.st, (const float*)a->M, a->ldm, a->G, a->ldg, g_mode, m, n, s.W(b, s.L.B32), bh, bl);
  else launch_pdl(k_form_b32<false>, grid, dim3(256), 0, s.st, (const float*)a->M, a->ldm, a->G, a->ldg, g_mode, m, n, s.W(b, s.L.B32), bh, bl);
  DION_CHECK_LAUNCH(c);
  return DION_OK;
}

// form_sum for every matrix of the chain: one launch when M and G share leading dimensions and alignment.
int form_sum_chain(StepCtx& s, const dion_matrix* const* list, bool pair) {
  dion_ctx* c = s.c;
  const dion_matrix* a0 = list[0];
  auto vec_ok = [](const dion_matrix* a) {
    return !((uintptr_t)a->M & 15) && a->ldm % 4 == 0 &&
           (a->g_dtype == DION_BF16 ? (!((uintptr_t)a->G & 7) && a->ldg % 4 == 0) : (!((uintptr_t)a->G & 15) && a->ldg % 4 == 0));
  };
  bool one = s.nb > 1 && s.nb <= GEMM_TAB_MAX && c->chain_batch;
  const bool vec = vec_ok(a0);
  for (int b = 1; b < s.nb && one; ++b)
    one = list[b]->ldm == a0->ldm && list[b]->ldg == a0->ldg && list[b]->g_dtype == a0->g_dtype && vec_ok(list[b]) == vec;
  if (!one) {
    for (int b = 0; b < s.nb; ++b) DION_TRY(form_sum(s, b, list[b], pair));
    return DION_OK;
  }
  const i64 m = a0->m, n = a0->n;
  ChainPtrs Ms, Gs;
  for (int b = 0; b < s.nb; ++b) { Ms.p[b] = list[b]->M; Gs.p[b] = list[b]->G; }
  const int g_mode = (a0->g_dtype == DION_BF16) ? ADD_BF16 : ADD_F32;
  __nv_bfloat16* bh = pair ? reinterpret_cast<__nv_bfloat16*>(s.ws + s.L.Bp) : nullptr;
  __nv_bfloat16* bl = pair ? bh + m * n : nullptr;
  const dim3 grid((unsigned)grid_for(c, m * n / 4), (unsigned)s.nb);
  if (vec) launch_pdl(k_form_b32_chain<true>, grid, dim3(256), 0, s.st, Ms, a0->ldm, Gs, a0->ldg, g_mode, m, n, s.ws + s.L.B32, bh, bl, s.wstride);
  else launch_pdl(k_form_b32_chain<false>, grid, dim3(256), 0, s.st, Ms, a0->ldm, Gs, a0->ldg, g_mode, m, n, s.ws + s.L.B32, bh, bl, s.wstride);
  DION_CHECK_LAUNCH(c);
  return DION_OK;
}

// The product itself: U (prow x r, dense) is split into the panel buffer `upair`; the pair of M + G must be in place.
int r_pairs(StepCtx& s, int b, const dion_matrix* a, bool tr, const float* U, float* upair, float* out, const int* skip,
            GemmArgs* defer = nullptr, bool split_done = false) {   // defer: the product is handed back instead of launched
  dion_ctx* c = s.c;
  const i64 m = a->m, n = a->n, r = a->r;
  const i64 prow = tr ? n : m, qrow = tr ? m : n;
  __nv_bfloat16* uh = reinterpret_cast<__nv_bfloat16*>(upair);
  __nv_bfloat16* ul = uh + prow * r;
  if (!split_done) {      // (the step splits U for the whole chain beforehand)
    launch_pdl(k_split_bf16, dim3((unsigned)grid_for(c, prow * r / 8)), dim3(256), 0, s.st, U, r, prow, r, uh, ul, skip);
    DION_CHECK_LAUNCH(c);
  }
  __nv_bfloat16* bh = reinterpret_cast<__nv_bfloat16*>(s.W(b, s.L.Bp));
  GemmArgs w = gemm_args();
  w.M = qrow; w.N = r; w.K = prow;
  w.ab16 = 1;
  w.A = (const float*)bh; w.A16lo = bh + m * n; w.a_si = tr ? n : 1; w.a_sk = tr ? 1 : n;
  w.B = (const float*)uh; w.B16lo = ul; w.b_sk = r; w.b_sn = 1;
  w.C = out; w.ldc = r; w.epi = EPI_STORE;
  w.skip_flag = skip;
  if (defer != nullptr) { *defer = w; return DION_OK; }
  return launch_gemm(s, w, b);
}

// The weight update X <- X - alpha F1 F2^T in fp32 mode on the tensor engine (F1: m x r with leading dimension
// ld1, F2: n x r with ld2; U Q^T, or Q U^T in the transposed form).  The update feeds nothing else, so its two
// factors are rounded to TF32 once (to nearest: unbiased) into `r1`, `r2` (scratch, dense) and the product takes
// one MMA per K step instead of three.  Returns false when the shape or the alignment does not qualify.
bool x_single_pass(const StepCtx& s, const dion_matrix* a, const float* F1, i64 ld1, const float* F2, i64 ld2) {
  const i64 m = a->m, n = a->n, r = a->r;
  return s.tensor && s.c->cfg.precision == DION_PREC_FP32 && m >= 128 && n >= 64 && r >= 64 && m % 4 == 0 &&
         n % 4 == 0 && r % 4 == 0 && !((uintptr_t)a->X & 15) && a->ldx % 4 == 0 && !((uintptr_t)F1 & 15) &&
         ld1 % 4 == 0 && !((uintptr_t)F2 & 15) && ld2 % 4 == 0;
}

// ... and with every dimension a multiple of 8 the rounded factors are IEEE half arrays instead: the same 11
// significant bits as TF32, read by one kind::f16 MMA per K step of 16 -- twice the MMA rate and half the operand
// bytes.  Both factors have unit-norm columns (U orthonormal, Q column-normalized), so their entries are at most 1;
// each is scaled by the power of two nearest the square root of its row count (entries around 1: far from half's
// subnormals, at most sqrt(2 rows) < 65504) and alpha takes the scales back exactly.
bool x_half(const dion_matrix* a) { return a->m % 8 == 0 && a->n % 8 == 0 && a->r % 8 == 0; }
float half_scale(i64 rows) { return exp2f(rintf(0.5f * log2f((float)rows))); }

// The error feedback M <- (M + G) - beta F1 F2^T in fp32 mode on the tensor engine (F1: m x r, F2: n x r; U R^T, or
// R U^T in the transposed form).  The product enters M scaled by beta = 1 - mu, so 16 significant bits in its factors
// are plenty (an error of ~1e-5 of the product, ~5e-7 of M): both factors are split once into bf16 pairs
// (hi, lo) in scratch (`p1`, `p2`: max(m,n) x r floats each) and the product takes three bf16 MMAs per K step, 1.3
// TF32 passes instead of three.  Otherwise the 3xTF32 / FMA product of the fp32 factors.
// sum32 != nullptr: M + G comes from scratch (C = sum32 - beta acc); else C = M + G - beta acc with the caller's G.
// ready1 / ready2: that factor's pair already sits in p1 / p2 (the step splits U for R).
bool ef_on_pairs(const StepCtx& s, const dion_matrix* a, const float* F1, i64 ld1, const float* F2, i64 ld2, const float* sum32) {
  const i64 m = a->m, n = a->n, r = a->r;
  return s.tensor && s.c->cfg.precision == DION_PREC_FP32 && m >= 128 && n >= 64 && r >= 64 && m % 8 == 0 &&
         n % 8 == 0 && r % 8 == 0 && !((uintptr_t)a->M & 15) && a->ldm % 4 == 0 && !((uintptr_t)F1 & 15) &&
         ld1 % 4 == 0 && !((uintptr_t)F2 & 15) && ld2 % 4 == 0 &&
         (sum32 != nullptr || (!((uintptr_t)a->G & 15) && a->ldg % ((a->g_dtype == DION_BF16) ? 8 : 4) == 0));
}

int ef_update(StepCtx& s, int b, const dion_matrix* a, const float* F1, i64 ld1, const float* F2, i64 ld2, float* p1,
              float* p2, const float* sum32, const int* skip, bool ready1 = false, bool ready2 = false,
              GemmArgs* defer = nullptr) {
  dion_ctx* c = s.c;
  const i64 m = a->m, n = a->n, r = a->r;
  GemmArgs e = gemm_args();
  e.M = m; e.N = n; e.K = r;
  const bool pairs = ef_on_pairs(s, a, F1, ld1, F2, ld2, sum32);
  if (pairs) {
    __nv_bfloat16* h1 = reinterpret_cast<__nv_bfloat16*>(p1);
    __nv_bfloat16* l1 = h1 + m * r;
    __nv_bfloat16* h2 = reinterpret_cast<__nv_bfloat16*>(p2);
    __nv_bfloat16* l2 = h2 + n * r;
    if (!ready1) {
      launch_pdl(k_split_bf16, dim3((unsigned)grid_for(c, m * r / 8)), dim3(256), 0, s.st, F1, ld1, m, r, h1, l1, skip);
      DION_CHECK_LAUNCH(c);
    }
    if (!ready2) {
      launch_pdl(k_split_bf16, dim3((unsigned)grid_for(c, n * r / 8)), dim3(256), 0, s.st, F2, ld2, n, r, h2, l2, skip);
      DION_CHECK_LAUNCH(c);
    }
    e.ab16 = 1;
    e.A = (const float*)h1; e.A16lo = l1; e.a_si = r; e.a_sk = 1;
    e.B = (const float*)h2; e.B16lo = l2; e.b_sk = 1; e.b_sn = r;
  } else {
    e.A = F1; e.a_si = ld1; e.a_sk = 1;
    e.B = F2; e.b_sk = 1; e.b_sn = ld2;
  }
  e.C = (float*)a->M; e.ldc = a->ldm;
  if (sum32 != nullptr) { e.epi = EPI_C2_SUB; e.C2 = sum32; e.ldc2 = n; e.c2_mode = ADD_F32; }
  else { e.epi = EPI_ADD2_SUB; e.C2 = a->G; e.ldc2 = a->ldg; e.c2_mode = (a->g_dtype == DION_BF16) ? ADD_BF16 : ADD_F32; }
  e.alpha = 1.f - c->cfg.mu;
  e.skip_flag = skip;
  if (defer != nullptr) { *defer = e; return DION_OK; }
  return launch_gemm(s, e, b);
}

int x_update(StepCtx& s, int b, const dion_matrix* a, const float* F1, i64 ld1, const float* F2, i64 ld2, float* r1,
             float* r2, float alpha, const int* skip, const float* alpha_dev = nullptr, GemmArgs* defer = nullptr,
             bool rounded = false) {   // rounded: r1 and r2 already hold the rounded factors
  dion_ctx* c = s.c;
  const i64 m = a->m, n = a->n, r = a->r;
  GemmArgs x = gemm_args();
  x.M = m; x.N = n; x.K = r;
  if (x_single_pass(s, a, F1, ld1, F2, ld2) && x_half(a)) {
    const float s1 = half_scale(m), s2 = half_scale(n);
    if (!rounded) {
      launch_pdl(k_round_f16, dim3((unsigned)grid_for(c, m * r / 8)), dim3(256), 0, s.st, F1, ld1, m, r, s1, reinterpret_cast<__half*>(r1), skip);
      DION_CHECK_LAUNCH(c);
      launch_pdl(k_round_f16, dim3((unsigned)grid_for(c, n * r / 8)), dim3(256), 0, s.st, F2, ld2, n, r, s2, reinterpret_cast<__half*>(r2), skip);
      DION_CHECK_LAUNCH(c);
    }
    x.ab16 = 1; x.f16 = 1;
    x.A = r1; x.a_si = r; x.a_sk = 1;
    x.B = r2; x.b_sk = 1; x.b_sn = r;
    alpha /= s1 * s2;       // (powers of two: exact)
  } else if (x_single_pass(s, a, F1, ld1, F2, ld2)) {
    if (!rounded) {
      launch_pdl(k_round_tf32, dim3((unsigned)grid_for(c, m * r / 4)), dim3(256), 0, s.st, F1, ld1, m, r, r1, skip);
      DION_CHECK_LAUNCH(c);
      launch_pdl(k_round_tf32, dim3((unsigned)grid_for(c, n * r / 4)), dim3(256), 0, s.st, F2, ld2, n, r, r2, skip);
      DION_CHECK_LAUNCH(c);
    }
    x.tf32x1 = 1;
    x.A = r1; x.a_si = r; x.a_sk = 1;
    x.B = r2; x.b_sk = 1; x.b_sn = r;
  } else {
    x.A = F1; x.a_si = ld1; x.a_sk = 1;
    x.B = F2; x.b_sk = 1; x.b_sn = ld2;
  }
  x.C = (float*)a->X; x.ldc = a->ldx; x.epi = EPI_SUB;
  x.alpha = alpha;
  x.alpha_dev = alpha_dev;      // graph replay: alpha = 1, the factor comes from the device scalar
  x.skip_flag = skip;
  if (defer != nullptr) { *defer = x; return DION_OK; }
  return launch_gemm(s, x, b);
}

// The launch chain of one Dion step (Algorithm 1 + 2) on `nb` matrices of identical
// (m, n, r), phase by phase.  Scratch must hold nb slices.
// x_scale != nullptr (graph capture, nb = 1, fp32 mode): the update's factor lr sqrt(m/n) is read from that device
// scalar and the step uses state slot `fixed_slot`.
int step_batch(dion_ctx* c, const dion_matrix* const* list, int nb, float lr, cudaStream_t st,
               const float* x_scale = nullptr, int fixed_slot = -1) {
  StepCtx s;
  const dion_matrix* a0 = list[0];
  DION_TRY(begin_step(c, a0, nb, st, &s, fixed_slot));
  const i64 m = a0->m, n = a0->n, r = a0->r;
  s.list = list;
  if (c->cfg.orth == DION_ORTH_RCQR) {
    const i64 panel_rows = a0->transposed ? n : m;
    for (int b = 0; b < nb; ++b) {
      const dion_matrix* a = list[b];
      if (a->sketch == nullptr || ((uintptr_t)a->sketch & 3)) return DION_ERR_INVALID;
      if (a->sketch_rows < r || a->sketch_rows > 2 * r || a->ld_sketch < panel_rows) return DION_ERR_SHAPE;
    }
  }

  // Standard form: the power iteration runs on B = M + G (panel P = B Q, m x r; Q is n x r).
  // Transposed form: it runs on B^T (panel P = B^T Q, n x r; Q is m x r), and the rank-r
  // products come out transposed: M <- B - (1 - mu) R U^T, X <- X - lr sqrt(m/n) Q U^T.
  const bool tr = a0->transposed != 0;
  const i64 prow = tr ? n : m;     // rows of the panel that is orthonormalized
  const i64 qrow = tr ? m : n;     // rows of R and Q
  const auto g_mode = [](const dion_matrix* a) { return (a->g_dtype == DION_BF16) ? ADD_BF16 : ADD_F32; };

  // bf16-operand mode on the tensor engine: bf16(M + G) is formed once per step and the four
  // products read bf16 arrays (B16, and the bf16 copies of Q, U, R) straight through TMA.
  bool d16 = s.tensor && c->cfg.precision == DION_PREC_BF16_OPERANDS && m % 8 == 0 && n % 8 == 0 && r % 8 == 0 &&
             m >= 128 && n >= 128 && r >= 64;
  for (int b = 0; b < nb && d16; ++b)
    if (((uintptr_t)list[b]->Q & 15) || (list[b]->ldq % 4)) d16 = false;
  auto bf = [&](int b, i64 off) { return reinterpret_cast<__nv_bfloat16*>(s.W(b, off)); };
  auto to_bf16 = [&](const float* src, i64 lds, i64 rows, i64 cols, __nv_bfloat16* out) -> int {
    launch_pdl(k_to_bf16, dim3((unsigned)(grid_for(c, rows * cols / 8))), dim3(256), 0, st, src, lds, rows, cols, out, nullptr);
    DION_CHECK_LAUNCH(c);
    return DION_OK;
  };

  // fp32 mode: M + G kept in scratch for P, R and the error feedback (see sum_in_scratch)
  const bool b32 = !d16 && s.tensor && s.L.B32 > 0;
  // ... R then runs on bf16 pairs of M + G and of U (three bf16 MMAs per K step: 1.3 TF32 passes instead of 3; the
  // product is accurate to ~1e-5, which is what Q <- ColNorm(R) and the error feedback need of it)
  const bool bpair = b32 && r_on_pairs(s, m, n, r);
  // ... and so does P where the orthonormalization is CholeskyQR2 and the matrix is large enough for the saving to
  // exceed the launches that stand by for the accurate product (see orthonormalize).  The rule looks at the matrix
  // alone, so that a grouped call computes what single calls compute.
  const bool ppair = bpair && (double)m * (double)n * (double)r >= P_PAIR_MIN_MNR &&
                     resolve_orth_for(c, r, (m < n) ? m : n, s.list != nullptr) == DION_ORTH_CHOLQR2;
  bool any_pair = false;

  // the large products: one GemmArgs per matrix, then one launch over the chain where that is possible
  std::vector<GemmArgs> group((size_t)nb);

  // P = (M + G) Q   (transposed form: (M + G)^T Q)
  const i64 pin_off = panel_offset(s, r, (m < n) ? m : n);
  bool q_copied = false;      // a dense copy of every Q of the chain sits in scratch (for the recomputation of P)
  {
  PhaseScope ps(c, st, DION_PHASE_P);
  // elementwise preparation for the whole chain: M + G (and its pair), the pair of Q where P takes pairs
  const float* srcs[MAX_CHAIN];
  i64 lds[MAX_CHAIN];
  if (b32) DION_TRY(form_sum_chain(s, list, bpair));
  const bool phalf = b32 && s.L.Bh > 0;
  bool p_half_ready = false;
  if (phalf) {      // the scaled half pairs of M + G and of Q, for the whole chain
    bool all_ok = true;
    for (int b = 0; b < nb; ++b) {
      all_ok = all_ok && !((uintptr_t)list[b]->Q & 15) && list[b]->ldq % 4 == 0 && list[b]->ldq == list[0]->ldq;
      srcs[b] = (const float*)list[b]->Q;
    }
    if (all_ok && nb <= GEMM_TAB_MAX) {
      i64 parts = (m * n / 4 + 2047) / 2048;
      if (parts > AMAX_PARTS) parts = AMAX_PARTS;
      __half* bh = reinterpret_cast<__half*>(s.ws + s.L.Bh);
      launch_pdl(k_absmax_partial, dim3((unsigned)parts, (unsigned)nb), dim3(256), 0, st, (const float*)(s.ws + s.L.B32), n, m, n,
                 s.ws + s.L.pmax, s.wstride, (const int*)nullptr, (i64)0);
      DION_CHECK_LAUNCH(c);
      launch_pdl(k_split_f16_scaled, dim3((unsigned)grid_for(c, m * n / 8), (unsigned)nb), dim3(256), 0, st,
                 (const float*)(s.ws + s.L.B32), n, m, n, (const float*)(s.ws + s.L.pmax), (int)parts, bh, bh + m * n,
                 s.ws + s.L.pmax + AMAX_PARTS, s.wstride, (const int*)nullptr, (i64)0, ldexpf(1.f, -13), (const float*)nullptr);
      DION_CHECK_LAUNCH(c);
      ChainPtrs t;
      for (int b = 0; b < nb; ++b) t.p[b] = srcs[b];
      __half* qh = reinterpret_cast<__half*>(s.ws + s.L.S16);
      launch_pdl(k_split_f16_fixed, dim3((unsigned)grid_for(c, qrow * r / 8), (unsigned)nb), dim3(256), 0, st, t, list[0]->ldq, qrow, r,
                 ldexpf(1.f, 13), qh, qh + qrow * r, s.wstride, (i64)0, (const int*)nullptr, (i64)0);
      DION_CHECK_LAUNCH(c);
      p_half_ready = true;
    }
  }
  bool q_split = false;
  if (b32 && ppair) {
    bool all_ok = true;
    for (int b = 0; b < nb; ++b) {
      all_ok = all_ok && !((uintptr_t)list[b]->Q & 15) && list[b]->ldq % 4 == 0;
      srcs[b] = (const float*)list[b]->Q; lds[b] = list[b]->ldq;
    }
    if (all_ok) { DION_TRY(split_chain(s, srcs, lds, qrow, r, s.L.S16, nullptr, s.L.Qc > 0 ? s.L.Qc : -1, &q_copied)); q_split = true; }
  }
  for (int b = 0; b < nb; ++b) {
    const dion_matrix* a = list[b];
    GemmArgs p = gemm_args();
    p.M = prow; p.N = r; p.K = qrow;
    if (d16) {
      const bool vec = !((uintptr_t)a->M & 15) && a->ldm % 4 == 0 &&
                       (a->g_dtype == DION_BF16 ? (!((uintptr_t)a->G & 15) && a->ldg % 8 == 0)
                                                : (!((uintptr_t)a->G & 15) && a->ldg % 4 == 0));
      const int grid = grid_for(c, m * n / 8);
      if (vec) launch_pdl(k_form_b16<true>, grid, dim3(256), 0, st, (const float*)a->M, a->ldm, a->G, a->ldg, g_mode(a), m, n, bf(b, s.L.B16));
      else launch_pdl(k_form_b16<false>, grid, dim3(256), 0, st, (const float*)a->M, a->ldm, a->G, a->ldg, g_mode(a), m, n, bf(b, s.L.B16));
      DION_CHECK_LAUNCH(c);
      DION_TRY(to_bf16((const float*)a->Q, a->ldq, qrow, r, bf(b, s.L.Q16)));
      p.ab16 = 1;
      p.A = (const float*)bf(b, s.L.B16); p.a_si = tr ? 1 : n; p.a_sk = tr ? n : 1;
      p.B = (const float*)bf(b, s.L.Q16); p.b_sk = r; p.b_sn = 1;
    } else if (b32 && ppair && !((uintptr_t)a->Q & 15) && a->ldq % 4 == 0) {
      __nv_bfloat16* qh = reinterpret_cast<__nv_bfloat16*>(s.W(b, s.L.S16));
      __nv_bfloat16* ql = qh + qrow * r;
      if (!q_split) {
        launch_pdl(k_split_bf16, dim3((unsigned)grid_for(c, qrow * r / 8)), dim3(256), 0, st, (const float*)a->Q, a->ldq, qrow, r, qh, ql,
                   (const int*)nullptr);
        DION_CHECK_LAUNCH(c);
      }
      __nv_bfloat16* bh = reinterpret_cast<__nv_bfloat16*>(s.W(b, s.L.Bp));
      p.ab16 = 1;
      p.A = (const float*)bh; p.A16lo = bh + m * n; p.a_si = tr ? 1 : n; p.a_sk = tr ? n : 1;
      p.B = (const float*)qh; p.B16lo = ql; p.b_sk = r; p.b_sn = 1;
      any_pair = true;
    } else if (p_half_ready) {
      __half* bh = reinterpret_cast<__half*>(s.W(b, s.L.Bh));
      __half* qh = reinterpret_cast<__half*>(s.W(b, s.L.S16));
      p.ab16 = 1; p.f16 = 1;
      p.A = (const float*)bh; p.A16lo = bh + m * n; p.a_si = tr ? 1 : n; p.a_sk = tr ? n : 1;
      p.B = (const float*)qh; p.B16lo = qh + qrow * r; p.b_sk = r; p.b_sn = 1;
      p.alpha_dev = s.W(b, s.L.pmax) + AMAX_PARTS;
    } else if (b32) {
      p.A = s.W(b, s.L.B32); p.a_si = tr ? 1 : n; p.a_sk = tr ? n : 1;
      p.B = (const float*)a->Q; p.b_sk = a->ldq; p.b_sn = 1;
    } else {
      p.A = (const float*)a->M; p.a_si = tr ? 1 : a->ldm; p.a_sk = tr ? a->ldm : 1;
      p.A2 = a->G; p.a2_si = tr ? 1 : a->ldg; p.a2_sk = tr ? a->ldg : 1; p.a2_mode = g_mode(a);
      p.B = (const float*)a->Q; p.b_sk = a->ldq; p.b_sn = 1;
    }
    p.C = s.W(b, pin_off); p.ldc = r; p.epi = EPI_STORE;
    // an ill-conditioned panel amplifies the error of P: use the accurate product there
    p.precise = (!d16 && resolve_orth(c, r, (m < n) ? m : n) == DION_ORTH_SHIFTED3) ? 1 : 0;
    group[b] = p;
  }
  DION_TRY(launch_gemm_group(s, group));
  }

  // U = Orthonormalize(P)
  i64 U_off = 0;
  {
  PhaseScope ps(c, st, DION_PHASE_ORTH);
  const std::function<int()> redo = [&]() -> int {
    std::vector<GemmArgs> again((size_t)nb);
    for (int b = 0; b < nb; ++b) {
      const dion_matrix* a = list[b];
      GemmArgs p = gemm_args();
      p.M = prow; p.N = r; p.K = qrow;
      p.A = s.W(b, s.L.B32); p.a_si = tr ? 1 : n; p.a_sk = tr ? n : 1;
      if (q_copied) { p.B = s.W(b, s.L.Qc); p.b_sk = r; p.b_sn = 1; }     // (the same values: one launch over the chain)
      else { p.B = (const float*)a->Q; p.b_sk = a->ldq; p.b_sn = 1; }
      p.C = s.W(b, pin_off); p.ldc = r; p.epi = EPI_STORE;
      p.skip_flag = s.OS(b) + OS_DONE;
      again[b] = p;
    }
    return launch_gemm_group(s, again);
  };
  s.in_orth = true;
  s.redo_p = any_pair ? &redo : nullptr;
  const int rc_orth = orthonormalize(s, prow, r, (m < n) ? m : n, pin_off, &U_off);
  s.redo_p = nullptr;
  s.in_orth = false;
  DION_TRY(rc_orth);
  }

  // R = (M + G)^T U   (transposed form: (M + G) U)
  {
  PhaseScope ps(c, st, DION_PHASE_R);
  const i64 other_off = (U_off == s.L.P0) ? s.L.P1 : s.L.P0;
  if (!d16 && bpair) {   // U as a bf16 pair in the other panel buffer, for the whole chain
    const float* srcs[MAX_CHAIN];
    i64 lds[MAX_CHAIN];
    for (int b = 0; b < nb; ++b) { srcs[b] = s.W(b, U_off); lds[b] = r; }
    DION_TRY(split_chain(s, srcs, lds, prow, r, other_off, s.os + OS_FAIL));
  }
  for (int b = 0; b < nb; ++b) {
    const dion_matrix* a = list[b];
    GemmArgs w = gemm_args();
    w.M = qrow; w.N = r; w.K = prow;
    if (d16) {
      DION_TRY(to_bf16(s.W(b, U_off), r, prow, r, bf(b, s.L.U16)));
      w.ab16 = 1;
      w.A = (const float*)bf(b, s.L.B16); w.a_si = tr ? n : 1; w.a_sk = tr ? 1 : n;
      w.B = (const float*)bf(b, s.L.U16); w.b_sk = r; w.b_sn = 1;
    } else if (bpair) {
      // U as a bf16 pair in the other panel buffer (the error feedback reuses it)
      DION_TRY(r_pairs(s, b, a, tr, s.W(b, U_off), s.W(b, other_off), s.W(b, s.L.R), s.OS(b) + OS_FAIL, &group[b], true));
      continue;
    } else if (b32) {
      w.A = s.W(b, s.L.B32); w.a_si = tr ? n : 1; w.a_sk = tr ? 1 : n;
      w.B = s.W(b, U_off); w.b_sk = r; w.b_sn = 1;
    } else {
      w.A = (const float*)a->M; w.a_si = tr ? a->ldm : 1; w.a_sk = tr ? 1 : a->ldm;
      w.A2 = a->G; w.a2_si = tr ? a->ldg : 1; w.a2_sk = tr ? 1 : a->ldg; w.a2_mode = g_mode(a);
      w.B = s.W(b, U_off); w.b_sk = r; w.b_sn = 1;
    }
    w.C = s.W(b, s.L.R); w.ldc = r; w.epi = EPI_STORE;
    group[b] = w;
  }
  DION_TRY(launch_gemm_group(s, group));
  }

  // M <- (M + G) - (1 - mu) U R^T   (transposed form: R U^T)
  {
  PhaseScope ps(c, st, DION_PHASE_EF);
  const i64 other_off = (U_off == s.L.P0) ? s.L.P1 : s.L.P0;
  bool ef_split = false;      // the factors' pairs are made for the whole chain when every matrix takes pairs
  if (!d16) {
    const float* srcs[MAX_CHAIN];
    i64 lds[MAX_CHAIN];
    bool all_pairs = true;
    for (int b = 0; b < nb; ++b) {
      const float* sum32 = b32 ? s.W(b, s.L.B32) : nullptr;
      all_pairs = all_pairs && (tr ? ef_on_pairs(s, list[b], s.W(b, s.L.R), r, s.W(b, U_off), r, sum32)
                                   : ef_on_pairs(s, list[b], s.W(b, U_off), r, s.W(b, s.L.R), r, sum32));
    }
    if (all_pairs) {
      for (int b = 0; b < nb; ++b) { srcs[b] = s.W(b, s.L.R); lds[b] = r; }
      DION_TRY(split_chain(s, srcs, lds, qrow, r, s.L.S16, s.os + OS_FAIL));
      if (!bpair) {
        for (int b = 0; b < nb; ++b) srcs[b] = s.W(b, U_off);
        DION_TRY(split_chain(s, srcs, lds, prow, r, other_off, s.os + OS_FAIL));
      }
      ef_split = true;
    }
  }
  for (int b = 0; b < nb; ++b) {
    const dion_matrix* a = list[b];
    if (d16) {
      GemmArgs e = gemm_args();
      e.M = m; e.N = n; e.K = r;
      DION_TRY(to_bf16(s.W(b, s.L.R), r, qrow, r, bf(b, s.L.R16)));
      e.ab16 = 1;
      e.A = (const float*)bf(b, tr ? s.L.R16 : s.L.U16); e.a_si = r; e.a_sk = 1;
      e.B = (const float*)bf(b, tr ? s.L.U16 : s.L.R16); e.b_sk = 1; e.b_sn = r;
      e.C = (float*)a->M; e.ldc = a->ldm;
      e.epi = EPI_ADD2_SUB; e.C2 = a->G; e.ldc2 = a->ldg; e.c2_mode = g_mode(a);
      e.alpha = 1.f - c->cfg.mu;
      e.skip_flag = s.OS(b) + OS_FAIL;
      group[b] = e;
      continue;
    }
    // the bf16 pairs of the two factors go to the other panel buffer and to their own buffer
    float* other = s.W(b, U_off == s.L.P0 ? s.L.P1 : s.L.P0);
    float* sbuf = s.W(b, s.L.S16);
    const float* Uf = s.W(b, U_off);
    const float* Rf = s.W(b, s.L.R);
    const float* sum32 = b32 ? s.W(b, s.L.B32) : nullptr;
    if (tr) DION_TRY(ef_update(s, b, a, Rf, r, Uf, r, sbuf, other, sum32, s.OS(b) + OS_FAIL, ef_split, bpair || ef_split, &group[b]));
    else DION_TRY(ef_update(s, b, a, Uf, r, Rf, r, other, sbuf, sum32, s.OS(b) + OS_FAIL, bpair || ef_split, ef_split, &group[b]));
  }
  DION_TRY(launch_gemm_group(s, group));
  }

  // Q <- ColNorm(R)
  {
  PhaseScope ps(c, st, DION_PHASE_COLNORM);
  DION_TRY(colnorm_chain(s, list, qrow, r));
  }

  // X <- X - lr sqrt(m/n) U Q^T   (transposed form: Q U^T)
  {
  PhaseScope ps(c, st, DION_PHASE_X);
  const float x_alpha = (x_scale != nullptr) ? 1.f : lr * sqrtf((float)((double)m / (double)n));
  const i64 other_off = (U_off == s.L.P0) ? s.L.P1 : s.L.P0;
  bool x_rounded = false;     // the rounded factors are made for the whole chain when every matrix takes the single pass
  if (!d16) {
    const float* srcs[MAX_CHAIN];
    i64 lds[MAX_CHAIN];
    bool all_one = true;
    for (int b = 0; b < nb; ++b) {
      const dion_matrix* a = list[b];
      all_one = all_one && (tr ? x_single_pass(s, a, (const float*)a->Q, a->ldq, s.W(b, U_off), r)
                               : x_single_pass(s, a, s.W(b, U_off), r, (const float*)a->Q, a->ldq));
    }
    if (all_one) {
      for (int b = 0; b < nb; ++b) { srcs[b] = s.W(b, U_off); lds[b] = r; }
      const bool half = x_half(a0);
      DION_TRY(round_chain(s, srcs, lds, prow, r, other_off, s.os + OS_FAIL, half ? half_scale(prow) : 0.f));
      for (int b = 0; b < nb; ++b) { srcs[b] = (const float*)list[b]->Q; lds[b] = list[b]->ldq; }
      DION_TRY(round_chain(s, srcs, lds, qrow, r, s.L.R, s.os + OS_FAIL, half ? half_scale(qrow) : 0.f));
      x_rounded = true;
    }
  }
  for (int b = 0; b < nb; ++b) {
    const dion_matrix* a = list[b];
    if (d16) {
      GemmArgs x = gemm_args();
      x.M = m; x.N = n; x.K = r;
      DION_TRY(to_bf16((const float*)a->Q, a->ldq, qrow, r, bf(b, s.L.Q16)));
      x.ab16 = 1;
      x.A = (const float*)bf(b, tr ? s.L.Q16 : s.L.U16); x.a_si = r; x.a_sk = 1;
      x.B = (const float*)bf(b, tr ? s.L.U16 : s.L.Q16); x.b_sk = 1; x.b_sn = r;
      x.C = (float*)a->X; x.ldc = a->ldx; x.epi = EPI_SUB;
      x.alpha = x_alpha;
      x.skip_flag = s.OS(b) + OS_FAIL;
      group[b] = x;
      continue;
    }
    // the rounded copies of the single-pass form go to the other panel buffer and to R's, both free by now
    float* other = s.W(b, U_off == s.L.P0 ? s.L.P1 : s.L.P0);
    float* rbuf = s.W(b, s.L.R);
    const float* Uf = s.W(b, U_off);
    const float* Qf = (const float*)a->Q;
    if (tr) DION_TRY(x_update(s, b, a, Qf, a->ldq, Uf, r, rbuf, other, x_alpha, s.OS(b) + OS_FAIL, x_scale, &group[b], x_rounded));
    else DION_TRY(x_update(s, b, a, Uf, r, Qf, a->ldq, other, rbuf, x_alpha, s.OS(b) + OS_FAIL, x_scale, &group[b], x_rounded));
  }
  DION_TRY(launch_gemm_group(s, group));
  launch_pdl(k_finish_step, dim3((unsigned)(nb)), dim3(1), 0, st, s.flag, c->dev_ints + 1);
  DION_CHECK_LAUNCH(c);
  }
  return DION_OK;
}

int step_one(dion_ctx* c, const dion_matrix* a, float lr, cudaStream_t st) {
  return step_batch(c, &a, 1, lr, st);
}

// ---- graph replay of launch-bound steps ----------------------------------------------------------------

__global__ void k_set_scalar(float* dst, float v) { *dst = v; }

void graphs_clear(dion_ctx* c) {
  for (auto& g : c->graphs) cudaGraphExecDestroy(g.exec);
  c->graphs.clear();
}

bool same_matrix(const dion_matrix& x, const dion_matrix& y) {
  return x.m == y.m && x.n == y.n && x.r == y.r && x.X == y.X && x.ldx == y.ldx && x.M == y.M && x.ldm == y.ldm &&
         x.G == y.G && x.ldg == y.ldg && x.g_dtype == y.g_dtype && x.Q == y.Q && x.ldq == y.ldq &&
         x.colnorm_out == y.colnorm_out && x.transposed == y.transposed && x.sketch == y.sketch &&
         x.sketch_rows == y.sketch_rows && x.ld_sketch == y.ld_sketch;
}

// A step on a small matrix is a chain of ~30 launches that take longer to issue than to run.  Such steps are
// captured once (on the context's own stream: the caller's may be the legacy stream, which cannot capture) and
// replayed as one graph launch into the caller's stream.
bool graph_eligible(const dion_ctx* c, const dion_matrix* a) {
  return c->graphs_on && !c->prof_on && c->cfg.precision == DION_PREC_FP32 && c->cfg.engine != DION_ENGINE_SIMT &&
         a->m * a->n <= GRAPH_MAX_ELEMS && a->r <= NBO_COLS && a->m >= 128 && a->n >= 64 && a->r >= 64 && a->m % 4 == 0 &&
         a->n % 4 == 0 && a->r % 4 == 0 && !((uintptr_t)a->X & 15) && a->ldx % 4 == 0;     // (the X update must take the tensor engine)
}

// Returns DION_OK when the step was launched as a graph, 1 when the caller should launch it plainly.
int step_graph(dion_ctx* c, const dion_matrix* a, float lr, cudaStream_t st) {
  dion_ctx::GraphEntry* e = nullptr;
  for (auto& g : c->graphs)
    if (same_matrix(g.key, *a)) { e = &g; break; }
  if (e == nullptr) {
    int index = -1;
    if ((int)c->graphs.size() < MAX_GRAPHS) {
      index = (int)c->graphs.size();
    } else {      // evict the least recently used one (its kernels are ordered before ours only on its own stream: wait)
      size_t lru = 0;
      for (size_t i = 1; i < c->graphs.size(); ++i)
        if (c->graphs[i].last_use < c->graphs[lru].last_use) lru = i;
      if (cudaDeviceSynchronize() != cudaSuccess) return DION_ERR_CUDA;
      cudaGraphExecDestroy(c->graphs[lru].exec);
      index = c->graphs[lru].index;
      c->graphs.erase(c->graphs.begin() + (long)lru);
    }
    const int64_t l0 = c->launches;
    cudaGraph_t graph = nullptr;
    if (cudaStreamBeginCapture(c->cap, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); return 1; }
    const int rc = step_batch(c, &a, 1, lr, c->cap, c->graph_scalars + index, MAX_FLAG_SLOTS - MAX_GRAPHS + index);
    const cudaError_t ce = cudaStreamEndCapture(c->cap, &graph);
    const int64_t nl = c->launches - l0;
    c->launches = l0;
    if (rc != DION_OK || ce != cudaSuccess || graph == nullptr) {
      cudaGetLastError();
      if (graph != nullptr) cudaGraphDestroy(graph);
      c->graphs_on = false;      // this chain does not capture here: plain launches from now on
      return 1;
    }
    cudaGraphExec_t exec = nullptr;
    const cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ie != cudaSuccess || exec == nullptr) { cudaGetLastError(); c->graphs_on = false; return 1; }
    c->graphs.push_back({*a, exec, nl, index, 0});
    e = &c->graphs.back();
  }
  e->last_use = ++c->graph_clock;
  k_set_scalar<<<1, 1, 0, st>>>(c->graph_scalars + e->index, lr * sqrtf((float)((double)a->m / (double)a->n)));
  if (cudaGetLastError() != cudaSuccess) return DION_ERR_CUDA;
  if (cudaGraphLaunch(e->exec, st) != cudaSuccess) { cudaGetLastError(); return DION_ERR_CUDA; }
  c->launches += e->launches + 1;
  return DION_OK;
}

// One Lazy-Dion step (Algorithm 6).
int lazy_one(dion_ctx* c, const dion_matrix* a, float lr, int refresh, cudaStream_t st) {
  StepCtx s;
  DION_TRY(begin_step(c, a, 1, st, &s));
  const i64 m = a->m, n = a->n, r = a->r;
  const int gmode = (a->g_dtype == DION_BF16) ? ADD_BF16 : ADD_F32;
  float* P0 = s.ws + s.L.P0;
  float* R = s.ws + s.L.R;
  const float* Mp = (const float*)a->M;
  // bf16-operand mode on the tensor engine: as in the Dion step, bf16(M + G) is formed once and the
  // products read bf16 arrays (B16, and bf16 copies of Q, T / W, ColNorm(W))
  const bool d16 = s.tensor && c->cfg.precision == DION_PREC_BF16_OPERANDS && m % 8 == 0 && n % 8 == 0 && r % 8 == 0 &&
                   m >= 128 && n >= 128 && r >= 64 && !((uintptr_t)a->Q & 15) && a->ldq % 4 == 0;
  auto bf = [&](i64 off) { return reinterpret_cast<__nv_bfloat16*>(s.ws + off); };
  auto to_bf16 = [&](const float* src, i64 lds, i64 rows, i64 cols, __nv_bfloat16* out) -> int {
    launch_pdl(k_to_bf16, dim3((unsigned)grid_for(c, rows * cols / 8)), dim3(256), 0, st, src, lds, rows, cols, out, nullptr);
    DION_CHECK_LAUNCH(c);
    return DION_OK;
  };
  // B Q -> out (m x r): the fused fp32 path, or B16 Q16
  auto b_times_q = [&](float* out, int precise) -> int {
    GemmArgs t = gemm_args();
    t.M = m; t.N = r; t.K = n;
    if (d16) {
      DION_TRY(to_bf16((const float*)a->Q, a->ldq, n, r, bf(s.L.Q16)));
      t.ab16 = 1;
      t.A = (const float*)bf(s.L.B16); t.a_si = n; t.a_sk = 1;
      t.B = (const float*)bf(s.L.Q16); t.b_sk = r; t.b_sn = 1;
    } else {
      t.A = Mp; t.a_si = a->ldm; t.a_sk = 1;
      t.A2 = a->G; t.a2_si = a->ldg; t.a2_sk = 1; t.a2_mode = gmode;
      t.B = (const float*)a->Q; t.b_sk = a->ldq; t.b_sn = 1;
      t.precise = precise;
    }
    t.C = out; t.ldc = r; t.epi = EPI_STORE;
    return launch_gemm(s, t);
  };
  if (d16) {
    const bool vec = !((uintptr_t)a->M & 15) && a->ldm % 4 == 0 && !((uintptr_t)a->G & 15) &&
                     a->ldg % ((a->g_dtype == DION_BF16) ? 8 : 4) == 0;
    const dim3 grid((unsigned)grid_for(c, m * n / 8));
    if (vec) launch_pdl(k_form_b16<true>, grid, dim3(256), 0, st, Mp, a->ldm, a->G, a->ldg, gmode, m, n, bf(s.L.B16));
    else launch_pdl(k_form_b16<false>, grid, dim3(256), 0, st, Mp, a->ldm, a->G, a->ldg, gmode, m, n, bf(s.L.B16));
    DION_CHECK_LAUNCH(c);
  }

  if (refresh) {
    // profiling: the whole refresh (SymPowerIter1) is booked as the ORTH phase
    PhaseScope ps_orth(c, st, DION_PHASE_ORTH);
    // T = (M + G) Q  (m x r), Z = (M + G)^T T (n x r), Q <- Orthonormalize(Z)
    const int precise = (resolve_orth(c, r, (m < n) ? m : n) == DION_ORTH_SHIFTED3) ? 1 : 0;
    DION_TRY(b_times_q(R, precise));
    GemmArgs z = gemm_args();
    z.M = n; z.N = r; z.K = m;
    if (d16) {
      DION_TRY(to_bf16(R, r, m, r, bf(s.L.U16)));
      z.ab16 = 1;
      z.A = (const float*)bf(s.L.B16); z.a_si = 1; z.a_sk = n;
      z.B = (const float*)bf(s.L.U16); z.b_sk = r; z.b_sn = 1;
    } else {
      z.A = Mp; z.a_si = 1; z.a_sk = a->ldm;
      z.A2 = a->G; z.a2_si = 1; z.a2_sk = a->ldg; z.a2_mode = gmode;
      z.B = R; z.b_sk = r; z.b_sn = 1;
      z.precise = precise;
    }
    const i64 pin_off = panel_offset(s, r, (m < n) ? m : n);
    z.C = s.ws + pin_off; z.ldc = r; z.epi = EPI_STORE;
    DION_TRY(launch_gemm(s, z));
    i64 V_off = 0;
    s.in_orth = true;
    const int rc_orth = orthonormalize(s, n, r, (m < n) ? m : n, pin_off, &V_off);
    s.in_orth = false;
    DION_TRY(rc_orth);
    const float* V = s.ws + V_off;
    // copy V into Q unless the round broke down
    const i64 total = n * r;
    int blocks = (int)((total + 255) / 256);
    if (blocks > 8 * c->sm_count) blocks = 8 * c->sm_count;
    launch_pdl(k_copy_panel, dim3((unsigned)(blocks)), dim3(256), 0, st, V, r, (float*)a->Q, a->ldq, n, r, s.flag, nullptr, 0);
    DION_CHECK_LAUNCH(c);
  }
  // W = (M + G) Q
  {
  PhaseScope ps(c, st, DION_PHASE_P);
  DION_TRY(b_times_q(R, 0));
  }
  // M <- (M + G) - (1 - mu) W Q^T
  {
  PhaseScope ps(c, st, DION_PHASE_EF);
  GemmArgs e = gemm_args();
  e.M = m; e.N = n; e.K = r;
  if (d16) {   // Q16 was written by b_times_q just above
    DION_TRY(to_bf16(R, r, m, r, bf(s.L.U16)));
    e.ab16 = 1;
    e.A = (const float*)bf(s.L.U16); e.a_si = r; e.a_sk = 1;
    e.B = (const float*)bf(s.L.Q16); e.b_sk = 1; e.b_sn = r;
  } else {
    e.A = R; e.a_si = r; e.a_sk = 1;
    e.B = (const float*)a->Q; e.b_sk = 1; e.b_sn = a->ldq;
  }
  e.C = (float*)a->M; e.ldc = a->ldm; e.epi = EPI_ADD2_SUB;
  e.C2 = a->G; e.ldc2 = a->ldg; e.c2_mode = gmode;
  e.alpha = 1.f - c->cfg.mu;
  e.skip_flag = s.flag;
  DION_TRY(launch_gemm(s, e));
  }
  // U = ColNorm(W)
  {
  PhaseScope ps(c, st, DION_PHASE_COLNORM);
  DION_TRY(colnorm(s, 0, R, m, r, P0, r, a->colnorm_out));
  }
  // X <- X - lr sqrt(m/n) U Q^T
  PhaseScope ps_x(c, st, DION_PHASE_X);
  GemmArgs x = gemm_args();
  x.M = m; x.N = n; x.K = r;
  if (d16) {
    DION_TRY(to_bf16(P0, r, m, r, bf(s.L.R16)));
    x.ab16 = 1;
    x.A = (const float*)bf(s.L.R16); x.a_si = r; x.a_sk = 1;
    x.B = (const float*)bf(s.L.Q16); x.b_sk = 1; x.b_sn = r;
  } else {
    x.A = P0; x.a_si = r; x.a_sk = 1;
    x.B = (const float*)a->Q; x.b_sk = 1; x.b_sn = a->ldq;
  }
  x.C = (float*)a->X; x.ldc = a->ldx; x.epi = EPI_SUB;
  x.alpha = lr * sqrtf((float)((double)m / (double)n));
  x.skip_flag = s.flag;
  DION_TRY(launch_gemm(s, x));
  launch_pdl(k_finish_step, dim3((unsigned)(1)), dim3(1), 0, st, s.flag, c->dev_ints + 1);
  DION_CHECK_LAUNCH(c);
  return DION_OK;
}

}  // namespace

extern "C" {

void dion_default_config(dion_config* cfg) {
  if (cfg == nullptr) return;
  cfg->mu = 0.95f;
  cfg->eps = 1e-8f;
  cfg->precision = DION_PREC_FP32;
  cfg->orth = DION_ORTH_AUTO;
  cfg->engine = DION_ENGINE_AUTO;
  cfg->device = 0;
  cfg->workspace_bytes = 0;
}

int dion_init(dion_ctx** out, const dion_config* cfg) {
  if (out == nullptr) return DION_ERR_INVALID;
  *out = nullptr;
  if (cfg == nullptr) return DION_ERR_INVALID;
  if (cfg->precision != DION_PREC_FP32 && cfg->precision != DION_PREC_BF16_OPERANDS) return DION_ERR_INVALID;
  if (cfg->orth < DION_ORTH_AUTO || cfg->orth > DION_ORTH_RCQR) return DION_ERR_INVALID;
  if (cfg->engine < DION_ENGINE_AUTO || cfg->engine > DION_ENGINE_TENSOR) return DION_ERR_INVALID;
  if (!(cfg->mu >= 0.f && cfg->mu <= 1.f) || !(cfg->eps >= 0.f)) return DION_ERR_INVALID;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device < 0 || cfg->device >= ndev) {
    cudaGetLastError();
    return DION_ERR_CUDA;
  }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return DION_ERR_CUDA;
  if (prop.major != 10) return DION_ERR_CUDA;  // built for sm_100a only
  if (cudaSetDevice(cfg->device) != cudaSuccess) return DION_ERR_CUDA;
  dion_ctx* c = new (std::nothrow) dion_ctx();
  if (c == nullptr) return DION_ERR_NOMEM;
  c->ws = nullptr; c->ws_bytes = 0; c->dev_ints = nullptr; c->flag_cursor = 0; c->launches = 0;
  c->prof_on = false; c->prof_used = 0;
  c->cfg = *cfg;
  c->sm_count = prop.multiProcessorCount;
  void* p = nullptr;
  if (cudaMalloc(&p, sizeof(int) * (8 + MAX_FLAG_SLOTS * OS_SLOT_INTS)) != cudaSuccess) { delete c; return DION_ERR_NOMEM; }
  c->dev_ints = (int*)p;
  if (cudaMemset(p, 0, sizeof(int) * (8 + MAX_FLAG_SLOTS * OS_SLOT_INTS)) != cudaSuccess) { cudaFree(p); delete c; return DION_ERR_CUDA; }
  if (configure_kernels() != DION_OK) { cudaFree(p); delete c; return DION_ERR_CUDA; }
  if (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); c->side = nullptr; }
  // graph replay of small steps: a capture stream and the scalars the graphs read; off if either cannot be had
  umma::pair_clusters(c->sm_count);      // (asked once per device, outside any capture)
  {
    void* gs = nullptr;
    if (cudaStreamCreateWithFlags(&c->cap, cudaStreamNonBlocking) == cudaSuccess &&
        cudaMalloc(&gs, sizeof(float) * MAX_GRAPHS) == cudaSuccess) {
      c->graph_scalars = (float*)gs;
      c->graphs_on = true;
    } else {
      cudaGetLastError();
      if (c->cap != nullptr) { cudaStreamDestroy(c->cap); c->cap = nullptr; }
    }
  }
  for (int i = 0; i < 32 && c->side != nullptr; ++i)
    if (cudaEventCreateWithFlags(&c->side_ev[i], cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError();
      cudaStreamDestroy(c->side);
      c->side = nullptr;      // no look-ahead: everything runs on the caller's stream
    }
  if (cfg->workspace_bytes > 0) {
    const int rc = ensure_ws(c, cfg->workspace_bytes);
    if (rc != DION_OK) { cudaFree(c->dev_ints); delete c; return rc; }
  }
  *out = c;
  return DION_OK;
}

size_t dion_workspace_bytes(const dion_ctx* ctx, int64_t m, int64_t n, int64_t r) {
  if (ctx == nullptr || m < 1 || n < 1 || r < 1 || r > m || r > n) return 0;
  return (size_t)make_layout(ctx, m, n, r).total * sizeof(float);
}

int dion_step(dion_ctx* ctx, const dion_matrix* a, float lr, void* cuda_stream) {
  if (ctx == nullptr) return DION_ERR_INVALID;
  DION_TRY(validate(a));
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  DION_TRY(ensure_ws(ctx, dion_workspace_bytes(ctx, a->m, a->n, a->r)));
  if (graph_eligible(ctx, a)) {
    const int rc = step_graph(ctx, a, lr, (cudaStream_t)cuda_stream);
    if (rc <= 0) return rc;
  }
  return step_one(ctx, a, lr, (cudaStream_t)cuda_stream);
}

int dion_step_grouped(dion_ctx* ctx, const dion_matrix* list, int count, float lr, void* cuda_stream) {
  if (ctx == nullptr || count < 0) return DION_ERR_INVALID;
  if (count == 0) return DION_OK;
  if (list == nullptr) return DION_ERR_INVALID;
  for (int i = 0; i < count; ++i) DION_TRY(validate(&list[i]));
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  // Matrices of identical (m, n, r) form a class (the paper's batch axis).  A class is
  // stepped in chains of up to `cap` matrices that share each small kernel launch of the
  // factorization; every matrix of a chain has its own scratch slice.
  const size_t budget = ctx->cfg.workspace_bytes > GROUP_SCRATCH_BYTES ? ctx->cfg.workspace_bytes : GROUP_SCRATCH_BYTES;
  std::vector<char> done((size_t)count, 0);
  std::vector<const dion_matrix*> chain;
  size_t need = 0;
  std::vector<std::vector<const dion_matrix*>> chains;
  for (int i = 0; i < count; ++i) {
    if (done[i]) continue;
    const size_t one = dion_workspace_bytes(ctx, list[i].m, list[i].n, list[i].r);
    size_t cap = one > 0 ? budget / one : 1;
    if (cap < 1) cap = 1;
    if (cap > MAX_CHAIN) cap = MAX_CHAIN;
    chain.clear();
    for (int j = i; j < count; ++j) {
      if (done[j] || list[j].m != list[i].m || list[j].n != list[i].n || list[j].r != list[i].r ||
          list[j].transposed != list[i].transposed || list[j].sketch_rows != list[i].sketch_rows) continue;
      done[j] = 1;
      chain.push_back(&list[j]);
      if (chain.size() == cap) { chains.push_back(chain); chain.clear(); }
    }
    if (!chain.empty()) chains.push_back(chain);
  }
  for (const auto& ch : chains) {
    const size_t b = dion_workspace_bytes(ctx, ch[0]->m, ch[0]->n, ch[0]->r) * ch.size();
    if (b > need) need = b;
  }
  DION_TRY(ensure_ws(ctx, need));
  for (const auto& ch : chains) DION_TRY(step_batch(ctx, ch.data(), (int)ch.size(), lr, (cudaStream_t)cuda_stream));
  return DION_OK;
}

int dion_lazy_step(dion_ctx* ctx, const dion_matrix* a, float lr, int refresh, void* cuda_stream) {
  if (ctx == nullptr) return DION_ERR_INVALID;
  DION_TRY(validate(a));
  if (a->transposed) return DION_ERR_INVALID;   // Algorithm 6 is built in the standard form only
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  DION_TRY(ensure_ws(ctx, dion_workspace_bytes(ctx, a->m, a->n, a->r)));
  return lazy_one(ctx, a, lr, refresh, (cudaStream_t)cuda_stream);
}

// ---- compressed data-parallel sync: the step in three calls --------------------------------

namespace {

int dp_check(dion_ctx* ctx, const dion_matrix* a, const void* p0, const void* p1, const int* flag) {
  if (ctx == nullptr || p0 == nullptr || p1 == nullptr || flag == nullptr) return DION_ERR_INVALID;
  DION_TRY(validate(a));
  if (a->transposed) return DION_ERR_INVALID;
  if (((uintptr_t)p0 & 15) || ((uintptr_t)p1 & 15) || ((uintptr_t)flag & 3)) return DION_ERR_ALIGN;
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  return ensure_ws(ctx, dion_workspace_bytes(ctx, a->m, a->n, a->r));
}

GemmArgs dp_b_product(const dion_matrix* a, bool transposed_b, const float* rhs, float* out) {
  const i64 m = a->m, n = a->n, r = a->r;
  GemmArgs g = gemm_args();
  g.M = transposed_b ? n : m; g.N = r; g.K = transposed_b ? m : n;
  g.A = (const float*)a->M; g.a_si = transposed_b ? 1 : a->ldm; g.a_sk = transposed_b ? a->ldm : 1;
  g.A2 = a->G; g.a2_si = transposed_b ? 1 : a->ldg; g.a2_sk = transposed_b ? a->ldg : 1;
  g.a2_mode = (a->g_dtype == DION_BF16) ? ADD_BF16 : ADD_F32;
  g.B = rhs; g.b_sk = r; g.b_sn = 1;
  g.C = out; g.ldc = r; g.epi = EPI_STORE;
  return g;
}

}  // namespace

int dion_dp_project(dion_ctx* ctx, const dion_matrix* a, float* P, int* dp_flag, void* cuda_stream) {
  DION_TRY(dp_check(ctx, a, P, P, dp_flag));
  StepCtx s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  DION_TRY(begin_step(ctx, a, 1, st, &s));
  if (cudaMemsetAsync(dp_flag, 0, sizeof(int), st) != cudaSuccess) return DION_ERR_CUDA;
  GemmArgs p = dp_b_product(a, false, (const float*)a->Q, P);
  p.b_sk = a->ldq;
  p.precise = (resolve_orth(ctx, a->r, (a->m < a->n) ? a->m : a->n) == DION_ORTH_SHIFTED3) ? 1 : 0;
  return launch_gemm(s, p, 0);
}

int dion_dp_factor(dion_ctx* ctx, const dion_matrix* a, float* PU, float* W, int* dp_flag, void* cuda_stream) {
  DION_TRY(dp_check(ctx, a, PU, W, dp_flag));
  if (ctx->cfg.orth == DION_ORTH_RCQR) return DION_ERR_UNSUPPORTED;
  StepCtx s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  DION_TRY(begin_step(ctx, a, 1, st, &s));
  const i64 m = a->m, n = a->n, r = a->r;
  dim3 grid((unsigned)grid_for(ctx, m * r), 1);
  const i64 pin_off = panel_offset(s, r, (m < n) ? m : n);
  launch_pdl(k_copy_block, grid, dim3(256), 0, st, PU, r, s.ws + pin_off, r, m, r, nullptr, 0);
  DION_CHECK_LAUNCH(ctx);
  i64 U_off = 0;
  s.in_orth = true;
  const int rc = orthonormalize(s, m, r, (m < n) ? m : n, pin_off, &U_off);
  s.in_orth = false;
  DION_TRY(rc);
  launch_pdl(k_copy_block, grid, dim3(256), 0, st, s.ws + U_off, r, PU, r, m, r, nullptr, 0);
  DION_CHECK_LAUNCH(ctx);
  launch_pdl(k_latch_flag, dim3((unsigned)(1)), dim3(1), 0, st, s.flag, dp_flag);      // a breakdown cancels dion_dp_finish
  DION_CHECK_LAUNCH(ctx);
  if (r_on_pairs(s, m, n, r)) {       // as dion_step: W on the bf16 pairs of M + G and U
    DION_TRY(form_sum(s, 0, a, true));
    return r_pairs(s, 0, a, false, PU, s.ws + s.L.P1, W, nullptr);
  }
  return launch_gemm(s, dp_b_product(a, true, PU, W), 0);
}

int dion_dp_finish(dion_ctx* ctx, const dion_matrix* a, const float* U, const float* W, const int* dp_flag,
                   float lr, void* cuda_stream) {
  DION_TRY(dp_check(ctx, a, U, W, dp_flag));
  StepCtx s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  DION_TRY(begin_step(ctx, a, 1, st, &s));
  const i64 m = a->m, n = a->n, r = a->r;
  // M <- (M + G) - (1 - mu) U W^T, with this rank's M and G (as in dion_step)
  DION_TRY(ef_update(s, 0, a, U, r, W, r, s.ws + s.L.P1, s.ws + s.L.S16, nullptr, dp_flag));
  DION_TRY(colnorm(s, 0, W, n, r, (float*)a->Q, a->ldq, a->colnorm_out, dp_flag));
  // X <- X - lr sqrt(m/n) U Q^T, as in dion_step (rounded copies in the two panel buffers of the scratch)
  DION_TRY(x_update(s, 0, a, U, r, (const float*)a->Q, a->ldq, s.ws + s.L.P1, s.ws + s.L.R,
                    lr * sqrtf((float)((double)m / (double)n)), dp_flag));
  launch_pdl(k_finish_step, dim3((unsigned)(1)), dim3(1), 0, st, dp_flag, ctx->dev_ints + 1);
  DION_CHECK_LAUNCH(ctx);
  return DION_OK;
}

// ---- 1D-sharded Dion (Algorithm 3): the per-rank pieces between its collectives -------------------

namespace {

int shard_check(dion_ctx* ctx, const dion_matrix* a, int64_t n_total, const void* p0, const void* p1, const int* flag) {
  if (ctx == nullptr || p0 == nullptr || p1 == nullptr || flag == nullptr) return DION_ERR_INVALID;
  DION_TRY(validate(a, true));
  if (a->transposed || n_total < a->n || a->r > n_total) return DION_ERR_INVALID;
  if (((uintptr_t)p0 & 15) || ((uintptr_t)p1 & 15) || ((uintptr_t)flag & 3)) return DION_ERR_ALIGN;
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  return ensure_ws(ctx, (size_t)make_layout(ctx, a->m, a->n, a->r).total * sizeof(float));
}

}  // namespace

int dion_shard_project(dion_ctx* ctx, const dion_matrix* a, int64_t n_total, float* P, int* flag, void* cuda_stream) {
  DION_TRY(shard_check(ctx, a, n_total, P, P, flag));
  StepCtx s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  DION_TRY(begin_step(ctx, a, 1, st, &s));
  if (cudaMemsetAsync(flag, 0, sizeof(int), st) != cudaSuccess) return DION_ERR_CUDA;
  GemmArgs p = dp_b_product(a, false, (const float*)a->Q, P);
  p.b_sk = a->ldq;
  p.precise = (resolve_orth(ctx, a->r, (a->m < n_total) ? a->m : n_total) == DION_ORTH_SHIFTED3) ? 1 : 0;
  return launch_gemm(s, p, 0);
}

int dion_orthonormalize(dion_ctx* ctx, int64_t m, int64_t r, int64_t n_total, float* PU, int* flag, void* cuda_stream) {
  if (ctx == nullptr || PU == nullptr || flag == nullptr) return DION_ERR_INVALID;
  if (m < 1 || n_total < 1 || r < 1 || r > m || r > n_total) return DION_ERR_SHAPE;
  if (((uintptr_t)PU & 15) || ((uintptr_t)flag & 3)) return DION_ERR_ALIGN;
  if (ctx->cfg.orth == DION_ORTH_RCQR) return DION_ERR_UNSUPPORTED;
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  dion_matrix shape;
  memset(&shape, 0, sizeof(shape));
  shape.m = m; shape.n = n_total; shape.r = r;
  DION_TRY(ensure_ws(ctx, (size_t)make_layout(ctx, m, n_total, r).total * sizeof(float)));
  StepCtx s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  DION_TRY(begin_step(ctx, &shape, 1, st, &s));
  const i64 sd = (m < n_total) ? m : n_total;
  const i64 pin_off = panel_offset(s, r, sd);
  dim3 grid((unsigned)grid_for(ctx, m * r), 1);
  launch_pdl(k_copy_block, grid, dim3(256), 0, st, (const float*)PU, r, s.ws + pin_off, r, m, r, nullptr, 0);
  DION_CHECK_LAUNCH(ctx);
  i64 U_off = 0;
  s.in_orth = true;
  const int rc = orthonormalize(s, m, r, sd, pin_off, &U_off);
  s.in_orth = false;
  DION_TRY(rc);
  launch_pdl(k_copy_block, grid, dim3(256), 0, st, (const float*)(s.ws + U_off), r, PU, r, m, r, nullptr, 0);
  DION_CHECK_LAUNCH(ctx);
  launch_pdl(k_latch_flag, dim3(1), dim3(1), 0, st, (const int*)s.flag, flag);
  DION_CHECK_LAUNCH(ctx);
  return DION_OK;
}

int dion_shard_factor(dion_ctx* ctx, const dion_matrix* a, int64_t n_total, const float* U, float* W, float* colsumsq,
                      const int* flag, void* cuda_stream) {
  DION_TRY(shard_check(ctx, a, n_total, U, W, flag));
  if (colsumsq == nullptr) return DION_ERR_INVALID;
  StepCtx s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  DION_TRY(begin_step(ctx, a, 1, st, &s));
  if (r_on_pairs(s, a->m, a->n, a->r)) {       // as dion_step: W on the bf16 pairs of M + G and U
    DION_TRY(form_sum(s, 0, a, true));
    DION_TRY(r_pairs(s, 0, a, false, U, s.ws + s.L.P1, W, flag));
  } else {
    GemmArgs w = dp_b_product(a, true, U, W);
    w.skip_flag = flag;
    DION_TRY(launch_gemm(s, w, 0));
  }
  int chunks; i64 per;
  colnorm_plan(a->n, a->r, ctx->sm_count, &chunks, &per);
  float* part = s.W(0, s.L.cn_part);
  dim3 grid((unsigned)((a->r + 127) / 128), (unsigned)chunks);
  launch_pdl(k_colsumsq_partial, grid, dim3(128), 0, st, (const float*)W, a->r, a->n, a->r, per, part, (const int*)flag, (i64)0);
  DION_CHECK_LAUNCH(ctx);
  launch_pdl(k_colsumsq_finish, dim3((unsigned)((a->r + 127) / 128)), dim3(128), 0, st, (const float*)part, chunks, a->r, colsumsq, flag);
  DION_CHECK_LAUNCH(ctx);
  return DION_OK;
}

int dion_shard_finish(dion_ctx* ctx, const dion_matrix* a, int64_t n_total, const float* U, const float* W,
                      const float* colsumsq, const int* flag, float lr, void* cuda_stream) {
  DION_TRY(shard_check(ctx, a, n_total, U, W, flag));
  if (colsumsq == nullptr) return DION_ERR_INVALID;
  StepCtx s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  DION_TRY(begin_step(ctx, a, 1, st, &s));
  const i64 m = a->m, n = a->n, r = a->r;
  // M <- (M + G) - (1 - mu) U W^T on the shard's columns
  DION_TRY(ef_update(s, 0, a, U, r, W, r, s.ws + s.L.P1, s.ws + s.L.S16, nullptr, flag));
  {   // Q <- W / (sqrt(colsumsq) + eps): the squared column norms are the all-reduced ones (one "chunk")
    int chunks; i64 per;
    colnorm_plan(n, r, ctx->sm_count, &chunks, &per);
    dim3 grid((unsigned)((r + 127) / 128), (unsigned)chunks);
    launch_pdl(k_colnorm_apply, grid, dim3(128), 0, st, W, r, n, r, per, 1, colsumsq, ctx->cfg.eps, (float*)a->Q, a->ldq,
               s.W(0, s.L.d), a->colnorm_out, ctx->dev_ints, (const int*)flag, (i64)0, ChainPtrs(), ChainPtrs());
    DION_CHECK_LAUNCH(ctx);
  }
  // X <- X - lr sqrt(m / n_total) U Q^T on the shard's columns
  DION_TRY(x_update(s, 0, a, U, r, (const float*)a->Q, a->ldq, s.ws + s.L.P1, s.ws + s.L.R,
                    lr * sqrtf((float)((double)m / (double)n_total)), flag));
  launch_pdl(k_finish_step, dim3(1), dim3(1), 0, st, flag, ctx->dev_ints + 1);
  DION_CHECK_LAUNCH(ctx);
  return DION_OK;
}

int dion_get_status(dion_ctx* ctx, void* cuda_stream, int* device_status, int* steps_skipped) {
  if (ctx == nullptr) return DION_ERR_INVALID;
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int host[2] = {0, 0};
  if (cudaMemcpyAsync(host, ctx->dev_ints, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DION_ERR_CUDA;
  if (cudaMemsetAsync(ctx->dev_ints, 0, sizeof(host), st) != cudaSuccess) return DION_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DION_ERR_CUDA;
  if (device_status != nullptr) *device_status = host[0];
  if (steps_skipped != nullptr) *steps_skipped = host[1];
  return DION_OK;
}

int dion_profile_enable(dion_ctx* ctx, int on) {
  if (ctx == nullptr) return DION_ERR_INVALID;
  ctx->prof_on = (on != 0);
  if (on) { ctx->prof_recs.clear(); ctx->prof_used = 0; }
  return DION_OK;
}

int dion_profile_read(dion_ctx* ctx, float* ms, int64_t* launches) {
  if (ctx == nullptr) return DION_ERR_INVALID;
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  float acc[DION_NUM_PHASES] = {0};
  int64_t nl[DION_NUM_PHASES] = {0};
  int rc = DION_OK;
  for (const auto& rec : ctx->prof_recs) {
    float t = 0.f;
    if (cudaEventSynchronize(rec.e1) != cudaSuccess || cudaEventElapsedTime(&t, rec.e0, rec.e1) != cudaSuccess) {
      rc = DION_ERR_CUDA;
      break;
    }
    acc[rec.phase] += t;
    nl[rec.phase] += rec.launches;
  }
  ctx->prof_recs.clear();
  ctx->prof_used = 0;
  for (int i = 0; i < DION_NUM_PHASES; ++i) {
    if (ms != nullptr) ms[i] = acc[i];
    if (launches != nullptr) launches[i] = nl[i];
  }
  return rc;
}

int dion_get_orth_rounds(dion_ctx* ctx, void* cuda_stream, int64_t* rounds) {
  if (ctx == nullptr || rounds == nullptr) return DION_ERR_INVALID;
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int host = 0;
  if (cudaMemcpyAsync(&host, ctx->dev_ints + 2, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DION_ERR_CUDA;
  if (cudaMemsetAsync(ctx->dev_ints + 2, 0, sizeof(int), st) != cudaSuccess) return DION_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DION_ERR_CUDA;
  *rounds = host;
  return DION_OK;
}

int dion_get_fallbacks(dion_ctx* ctx, void* cuda_stream, int64_t* fallbacks) {
  if (ctx == nullptr || fallbacks == nullptr) return DION_ERR_INVALID;
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int host = 0;
  if (cudaMemcpyAsync(&host, ctx->dev_ints + 3, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DION_ERR_CUDA;
  if (cudaMemsetAsync(ctx->dev_ints + 3, 0, sizeof(int), st) != cudaSuccess) return DION_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DION_ERR_CUDA;
  *fallbacks = host;
  return DION_OK;
}

int64_t dion_launch_count(const dion_ctx* ctx) { return ctx == nullptr ? 0 : ctx->launches; }

void dion_destroy(dion_ctx* ctx) {
  if (ctx == nullptr) return;
  cudaSetDevice(ctx->cfg.device);
  cudaDeviceSynchronize();
  graphs_clear(ctx);
  if (ctx->graph_scalars != nullptr) cudaFree(ctx->graph_scalars);
  if (ctx->cap != nullptr) cudaStreamDestroy(ctx->cap);
  if (ctx->ws != nullptr) cudaFree(ctx->ws);
  if (ctx->dev_ints != nullptr) cudaFree(ctx->dev_ints);
  for (cudaEvent_t e : ctx->prof_pool) cudaEventDestroy(e);
  for (int i = 0; i < 32; ++i)
    if (ctx->side_ev[i] != nullptr) cudaEventDestroy(ctx->side_ev[i]);
  if (ctx->side != nullptr) cudaStreamDestroy(ctx->side);
  delete ctx;
}

const char* dion_strerror(int code) {
  switch (code) {
    case DION_OK: return "ok";
    case DION_ERR_INVALID: return "invalid argument";
    case DION_ERR_SHAPE: return "bad shape, rank or leading dimension";
    case DION_ERR_ALIGN: return "misaligned pointer";
    case DION_ERR_ALIAS: return "arrays overlap";
    case DION_ERR_NOMEM: return "out of device memory";
    case DION_ERR_CUDA: return "CUDA error or no sm_100 device";
    case DION_ERR_UNSUPPORTED: return "shape not supported by the requested engine";
    case DION_ERR_TOO_LARGE: return "shape needs more scratch than the built-in array of dion_step_noalloc holds";
    default: return "unknown error";
  }
}

}  // extern "C"

// ---------------------------------------------------------------------------
// dion_step_noalloc: the same step with its scratch in a built-in device array.
// ---------------------------------------------------------------------------

namespace {

constexpr size_t NOALLOC_SCRATCH_BYTES = (size_t)24 << 20;  // 24 MiB, resident on every device that loads the library
constexpr size_t NOALLOC_INT_BYTES = 256;                   // status word, counters and one step slot
constexpr int NOALLOC_MAX_DEVICES = 64;

// Scratch of dion_step_noalloc.  In host code this name is only a handle for
// cudaGetSymbolAddress; the device address is looked up once per device below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

struct NoallocDevice {
  std::atomic<bool> ready;
  unsigned char* base;
  int sm_count;
};
NoallocDevice g_noalloc_dev[NOALLOC_MAX_DEVICES];
std::mutex g_noalloc_mutex;

template <typename K>
bool touch_kernel(K kernel) {
  cudaFuncAttributes fa;
  if (cudaFuncGetAttributes(&fa, kernel) != cudaSuccess) { cudaGetLastError(); return false; }
  return true;
}

// With lazy module loading a kernel's code is loaded at its first use, which may allocate device memory.
// Asking for the attributes of every kernel the launch chain can reach loads them all at set-up (the
// tensor-core variants are covered by configure_kernels, which sets an attribute on each).
bool preload_kernels() {
  bool ok = true;
  ok = ok && touch_kernel(k_gemm_simt<128, 128, 8, 8, 8>) && touch_kernel(k_gemm_simt<64, 64, 16, 4, 4>);
  ok = ok && touch_kernel(k_splitk_reduce) && touch_kernel(k_round_begin) && touch_kernel(k_potrf_diag);
  ok = ok && touch_kernel(k_chol_step) && touch_kernel(k_inv_finish) && touch_kernel(k_round_end) && touch_kernel(k_tiny_cholqr2);
  ok = ok && touch_kernel(k_probe_y) && touch_kernel(k_probe_y4) && touch_kernel(k_probe_w) && touch_kernel(k_probe_decide) && touch_kernel(k_reset_rounds);
  ok = ok && touch_kernel(k_orth_finish) && touch_kernel(k_cgs_fallback) && touch_kernel(k_copy_block);
  ok = ok && touch_kernel(k_colsumsq_partial) && touch_kernel(k_colnorm_apply) && touch_kernel(k_copy_panel);
  ok = ok && touch_kernel(k_latch_flag) && touch_kernel(k_finish_step) && touch_kernel(k_hh_reflector);
  ok = ok && touch_kernel(k_hh_apply) && touch_kernel(k_set_identity) && touch_kernel(k_sign_fix);
  ok = ok && touch_kernel(k_form_b16<true>) && touch_kernel(k_form_b16<false>) && touch_kernel(k_form_b32<true>);
  ok = ok && touch_kernel(k_form_b32<false>) && touch_kernel(k_to_bf16) && touch_kernel(k_round_tf32);
  ok = ok && touch_kernel(k_split_bf16);
  return ok;
}

// First use on the current device: resolve the array's device address and read the
// device attributes.  No allocation; must not run inside a stream capture.
int noalloc_setup(int device, NoallocDevice** out) {
  if (device < 0 || device >= NOALLOC_MAX_DEVICES) return DION_ERR_INVALID;
  NoallocDevice* d = &g_noalloc_dev[device];
  if (!d->ready.load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (d->ready.load(std::memory_order_relaxed)) { *out = d; return DION_OK; }
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
      cudaGetLastError();
      return DION_ERR_CUDA;
    }
    if (major != 10) return DION_ERR_CUDA;
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError();
      return DION_ERR_CUDA;
    }
    if (configure_kernels() != DION_OK || !preload_kernels()) return DION_ERR_CUDA;
    d->base = (unsigned char*)ptr;
    d->sm_count = sms;
    d->ready.store(true, std::memory_order_release);
  }
  *out = d;
  return DION_OK;
}

}  // namespace

extern "C" int dion_step_noalloc(const dion_matrix* a, float lr, float mu, float eps, void* cuda_stream) {
  DION_TRY(validate(a));
  if (!(mu >= 0.f && mu <= 1.f) || !(eps >= 0.f)) return DION_ERR_INVALID;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return DION_ERR_CUDA; }
  NoallocDevice* nd = nullptr;
  DION_TRY(noalloc_setup(device, &nd));

  // A context that lives on the host stack for this call only and points at the
  // built-in array: the launch chain is the one dion_step runs.
  dion_ctx c;
  dion_default_config(&c.cfg);
  c.cfg.mu = mu;
  c.cfg.eps = eps;
  c.cfg.device = device;
  c.sm_count = nd->sm_count;
  c.dev_ints = (int*)nd->base;
  c.ws = (float*)(nd->base + NOALLOC_INT_BYTES);
  c.ws_bytes = NOALLOC_SCRATCH_BYTES - NOALLOC_INT_BYTES;
  c.flag_cursor = 0;
  c.launches = 0;
  c.prof_on = false;
  c.prof_used = 0;
  c.form_sum = false;
  const size_t need = (size_t)make_layout(&c, a->m, a->n, a->r).total * sizeof(float);
  if (need > c.ws_bytes) return DION_ERR_TOO_LARGE;
  // The array keeps what the previous call left: clear the status word and counters.
  // (The step's own slot is cleared by the launch chain.)
  if (cudaMemsetAsync(c.dev_ints, 0, 8 * sizeof(int), (cudaStream_t)cuda_stream) != cudaSuccess) return DION_ERR_CUDA;
  return step_one(&c, a, lr, (cudaStream_t)cuda_stream);
}

extern "C" size_t dion_noalloc_scratch_limit(void) { return NOALLOC_SCRATCH_BYTES - NOALLOC_INT_BYTES; }

// ---------------------------------------------------------------------------
// Internal test hook (dion_internal.h)
// ---------------------------------------------------------------------------
// Test hook: the orthogonality estimate of the most recent step's CholeskyQR2 check (first matrix of the chain).
extern "C" int dion_debug_orth_measure(dion_ctx* ctx, void* cuda_stream, float* estimate) {
  if (ctx == nullptr || estimate == nullptr) return DION_ERR_INVALID;
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return DION_ERR_CUDA;
  const int slot = (ctx->flag_cursor + MAX_FLAG_SLOTS - 1) % MAX_FLAG_SLOTS;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaMemcpyAsync(estimate, ctx->dev_ints + 8 + (i64)slot * OS_SLOT_INTS + OS_MAXDEV, sizeof(float), cudaMemcpyDeviceToHost, st) !=
          cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return DION_ERR_CUDA;
  return DION_OK;
}

extern "C" int dion_debug_chain_batch(dion_ctx* ctx, int on) {
  if (ctx == nullptr) return DION_ERR_INVALID;
  ctx->chain_batch = on != 0;
  graphs_clear(ctx);
  return DION_OK;
}

extern "C" int dion_debug_gemm(int engine, int precision, const dion_debug_gemm_args* a, float* part,
                               int64_t part_floats, int* status, void* cuda_stream) {
  if (a == nullptr || status == nullptr) return DION_ERR_INVALID;
  int device = 0, sms = 0;
  if (cudaGetDevice(&device) != cudaSuccess) return DION_ERR_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return DION_ERR_CUDA;
  if (configure_kernels() != DION_OK) return DION_ERR_CUDA;
  GemmArgs g = gemm_args();
  g.M = a->M; g.N = a->N; g.K = a->K;
  g.A = a->A; g.a_si = a->a_si; g.a_sk = a->a_sk;
  g.A2 = a->A2; g.a2_si = a->a2_si; g.a2_sk = a->a2_sk; g.a2_mode = a->a2_mode;
  g.B = a->B; g.b_sk = a->b_sk; g.b_sn = a->b_sn;
  g.C = a->C; g.ldc = a->ldc; g.epi = a->epi;
  g.C2 = a->C2; g.ldc2 = a->ldc2; g.c2_mode = a->c2_mode;
  g.alpha = a->alpha; g.tri = a->tri; g.klimit = a->klimit; g.precise = a->precise; g.ab16 = a->ab16; g.tf32x1 = a->tf32x1; g.f16 = a->f16;
  g.A16lo = a->A16lo; g.B16lo = a->B16lo;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (engine == DION_ENGINE_TENSOR) {
    const int rc = umma_try_launch(g, precision, sms, part, part_floats, status, st, a->variant);
    if (rc > 0) return DION_OK;
    return rc < 0 ? rc : DION_ERR_UNSUPPORTED;
  }
  dion_ctx c;
  dion_default_config(&c.cfg);
  c.sm_count = sms; c.launches = 0; c.prof_on = false; c.prof_used = 0;
  return launch_gemm_simt(&c, g, st, part, part_floats, false);
}

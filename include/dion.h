/*
 * dion.h -- C-ABI of the B200-native (sm_100a) single-device Dion update step.
 *
 * The library implements the unsharded Dion rule of "Dion: Distributed
 * Orthonormalized Updates" (Algorithm 1 line 3 + Algorithm 2) for one
 * matrix-valued parameter X (m x n, m = rows = "out" dimension |I|, n = columns
 * = "in" dimension |J|) with gradient G, momentum M and warm-start right factor
 * Q (the paper's V, n x r):
 *
 *     B  = M + G                               Alg. 2, line 1
 *     P  = B Q                                 PowerIter1, line 1
 *     U  = Orthonormalize(P)                   PowerIter1, line 3; Section 3.2
 *     R  = B^T U                               PowerIter1, line 4  (the paper's W)
 *     M <- B - (1 - mu) U R^T                  Alg. 2, line 3; Eq. 1 (error feedback)
 *     Q <- ColNorm(R)                          Alg. 2, line 4
 *     X <- X - lr * sqrt(m/n) * U Q^T          Alg. 2, lines 5-6; Alg. 1, line 3
 *
 * Orthonormalize returns the thin-QR orthonormal factor whose triangular factor
 * has a positive diagonal.  ColNorm divides column j by (||column j||_2 + eps).
 *
 * General conventions
 *   - Every matrix pointer is a DEVICE pointer owned by the caller; matrices are
 *     dense row-major with a leading dimension given in ELEMENTS.
 *   - X, M, Q are updated in place; G is never written.  No two arrays of one
 *     matrix may overlap.
 *   - All step calls are asynchronous on the CUDA stream passed in (a
 *     cudaStream_t cast to void*; NULL = the legacy default stream) and never
 *     synchronise.  Device-side problems (Cholesky breakdown, non-finite pivot)
 *     are latched in a status word read by dion_get_status.  Work issued after
 *     a call on the same stream sees its results.  Inside a call the library
 *     may run part of the orthonormalization on a second stream of its own,
 *     forked from and joined back to the caller's stream with events; nothing
 *     of a call is left running outside that order.
 *   - A context's scratch is shared by its calls: two calls on one context must
 *     not overlap on the GPU (issue them on one stream or order them with
 *     events); use one context per concurrent stream.
 *   - The context owns only scratch memory (P/U, R, Gram and triangular factors,
 *     column norms, flags).  It grows on demand with cudaMalloc, which
 *     synchronises; after the first call with the largest shapes, or when
 *     dion_config.workspace_bytes was large enough, no call allocates.
 *   - Every function returns DION_OK (0) or a negative DION_ERR_* code; nothing
 *     is printed, thrown or aborted.
 *   - There is no CPU fallback: on a machine without a usable sm_100 device
 *     dion_init fails with DION_ERR_CUDA.
 */
#ifndef DION_H_
#define DION_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dion_ctx dion_ctx; /* opaque; owns scratch memory only */

typedef enum { DION_F32 = 0, DION_BF16 = 1 } dion_dtype;

/* Arithmetic of the four large contractions (P, R, U R^T, U Q^T); accumulation is fp32 everywhere.
 * DION_PREC_FP32:           X, M and Q stay within 1e-4 (relative, Frobenius) of the rule evaluated in float64
 *                           wherever the rule itself is that well determined.  On the FMA engine every product is
 *                           fp32.  On the tensor cores each product runs at the cheapest arithmetic that keeps
 *                           the bound: P with 22 significant bits (3-term TF32 split), or, on large matrices, with
 *                           16 bits first (pairs of bf16 arrays) and again with 22 when the orthonormalization's
 *                           probe finds the panel ill conditioned; R and U R^T with 16 bits (bf16 pairs, ~1e-5 of
 *                           the product; U R^T enters M scaled by 1 - mu); U Q^T with 11 bits on factors rounded
 *                           to nearest (3e-4 of the update, 3e-6 of X).
 * DION_PREC_BF16_OPERANDS:  operands rounded to bf16 (M + G is added in fp32, then rounded); 3e-2 on X, M, Q.
 * The products inside Orthonormalize carry 22 significant bits in both modes.          */
typedef enum { DION_PREC_FP32 = 0, DION_PREC_BF16_OPERANDS = 1 } dion_precision;

/* Orthonormalize (Section 3.2 and the appendix on Cholesky QR).
 * DION_ORTH_AUTO:        CholeskyQR2 when 4 r <= min(m, n), else the adaptive rounds.
 * DION_ORTH_CHOLQR2:     two rounds of Cholesky QR (cond(P) up to about 4e3).  A pivot that
 *                        is not positive is the paper's "CQR failure ... fall back to QR"
 *                        (appendix on Cholesky QR): the library keeps the panel and, in the
 *                        same call and without a host round trip, one more launch
 *                        orthonormalizes it column by column (classical Gram-Schmidt twice:
 *                        the same thin-QR factor); that launch returns at once when no
 *                        pivot failed.  Counted by dion_get_fallbacks.  Only a panel that
 *                        is rank deficient to fp32 accuracy (a column shrinking below 2e-6
 *                        of its norm) still cancels the step (DION_STATUS_BREAKDOWN).
 *                        Before the second round the first round's result U1 is measured on the
 *                        device (a randomized estimate of |U1^T U1 - I|_F from two passes over the
 *                        panel; the exact value for a panel of at most 512 rows and 64 columns, whose
 *                        whole orthonormalization is one launch); if it is orthonormal to 3e-5 per
 *                        column the second round is skipped (well-conditioned panels).
 * DION_ORTH_SHIFTED3:    adaptive Cholesky QR rounds for ill-conditioned panels such as
 *                        full rank: a column whose pivot falls below 1e-4 of its
 *                        squared norm is deflated, so a round cannot break down and
 *                        cuts cond(P) by up to ~100; rounds repeat (at most 6) until one sees a
 *                        well-conditioned panel, one more round then finishes.  The
 *                        decision is taken on the device; unused rounds are skipped.
 * DION_ORTH_HOUSEHOLDER: Householder QR (slow, most robust).
 * DION_ORTH_RCQR:        randomized Cholesky QR, the paper's Distributed-Orthonormalize
 *                        (Algorithm 4) on one device: with the caller's sketching matrix S
 *                        (dion_matrix.sketch), R1 = triangular factor of QR(S P), B = P R1^-1,
 *                        R2 = Cholesky(B^T B), U = B R2^-1.  The QR of the small sketch is done
 *                        by the deflating Cholesky QR rounds (R1 is never formed: each round's
 *                        triangular factor is applied to the sketch and to P at once), so the
 *                        Gram matrices of an ill-conditioned panel are taken from the sketch
 *                        rows only.  dion_lazy_step treats it as DION_ORTH_AUTO.           */
typedef enum {
  DION_ORTH_AUTO = 0,
  DION_ORTH_CHOLQR2 = 1,
  DION_ORTH_SHIFTED3 = 2,
  DION_ORTH_HOUSEHOLDER = 3,
  DION_ORTH_RCQR = 4
} dion_orth;

/* Which kernels carry the contractions.
 * DION_ENGINE_AUTO:   tensor cores (tcgen05) where the shape allows, else SIMT.
 * DION_ENGINE_SIMT:   fp32 FMA kernels only (any shape).
 * DION_ENGINE_TENSOR: tensor cores; shapes they cannot take are an error.      */
typedef enum { DION_ENGINE_AUTO = 0, DION_ENGINE_SIMT = 1, DION_ENGINE_TENSOR = 2 } dion_engine;

enum {
  DION_OK = 0,
  DION_ERR_INVALID = -1,    /* NULL pointer, bad enum, count < 0, ...              */
  DION_ERR_SHAPE = -2,      /* m, n < 1, r outside [1, min(m, n)], ld too small   */
  DION_ERR_ALIGN = -3,      /* a pointer is not aligned to its element size x 4   */
  DION_ERR_ALIAS = -4,      /* two arrays of one matrix overlap                   */
  DION_ERR_NOMEM = -5,      /* scratch allocation failed                          */
  DION_ERR_CUDA = -6,       /* a CUDA runtime call failed, or no sm_100 device    */
  DION_ERR_UNSUPPORTED = -7, /* the requested engine cannot take this shape       */
  DION_ERR_TOO_LARGE = -8    /* dion_step_noalloc: the shape needs more scratch than
                                the library's built-in array holds                 */
};

/* Bits of the device status word (dion_get_status). */
enum {
  DION_STATUS_BREAKDOWN = 1,  /* the panel was rank deficient (a Cholesky pivot <= 0 that the
                                 fallback could not cure either): the step that saw it left
                                 X, M and Q unchanged                              */
  DION_STATUS_NONFINITE = 2,  /* NaN or Inf in M, G or Q (seen in the trace of the panel's Gram
                                 matrix: the step is cancelled), or in a column norm of R */
  DION_STATUS_TIMEOUT = 4,    /* a bounded device-side wait ran out                */
  DION_STATUS_ILLCOND = 8     /* the adaptive rounds ran out before the panel was seen
                                 well conditioned; the result may be less accurate  */
};

typedef struct {
  float mu;               /* momentum / error-feedback coefficient, beta = 1 - mu (paper: beta = 0.05) */
  float eps;              /* ColNorm epsilon (1e-8)                                                    */
  int precision;          /* dion_precision                                                            */
  int orth;               /* dion_orth                                                                 */
  int engine;             /* dion_engine                                                               */
  int device;             /* CUDA device ordinal                                                       */
  size_t workspace_bytes; /* scratch to reserve at init; 0 = grow on demand                            */
} dion_config;

/* One matrix parameter and its optimizer state (Algorithm 1: "states M, V"). */
typedef struct {
  int64_t m, n, r;      /* 1 <= r <= min(m, n)                                       */
  void* X;              /* fp32, m x n, in/out                                       */
  int64_t ldx;
  void* M;              /* fp32, m x n, in/out (momentum / error-feedback buffer)    */
  int64_t ldm;
  const void* G;        /* g_dtype, m x n, read only                                 */
  int64_t ldg;
  int g_dtype;          /* dion_dtype                                                */
  void* Q;              /* fp32, n x r, in/out (right factor; any full-column-rank start) */
  int64_t ldq;
  float* colnorm_out;   /* optional: r floats, the column norms of R (estimates of the
                           leading singular values of B); may be NULL                */
  int transposed;       /* 0: standard form.  1: transposed form (Section 4.3, "other
                           variants": the power iteration runs on M^T): Q is m x r,
                             P = B^T Q (n x r),  U = Orthonormalize(P),  R = B U (m x r),
                             M <- B - (1 - mu) R U^T,  Q <- ColNorm(R),
                             X <- X - lr * sqrt(m/n) * Q U^T.
                           This is the standard step applied to X^T, M^T, G^T with the
                           arrays left in place; the factor sqrt(m/n) stays that of the
                           stored m x n parameter (rows = "out"), so both forms scale
                           the update alike.  It puts the orthonormalized panel on the
                           n side: cheaper when m > n.  dion_lazy_step rejects it.   */
  const void* sketch;   /* DION_ORTH_RCQR only (else ignored, may be NULL): the sketching
                           matrix S of Algorithm 4, fp32, sketch_rows x p row-major, where
                           p = m (n in the transposed form) is the number of rows of the
                           panel; read only.  The paper draws 1.25 r Gaussian rows; U does
                           not depend on S in exact arithmetic.                      */
  int64_t sketch_rows;  /* r <= sketch_rows <= 2 r                                   */
  int64_t ld_sketch;    /* >= p                                                      */
} dion_matrix;

/* Fill *cfg with the defaults: mu 0.95, eps 1e-8, fp32, AUTO, AUTO, device 0, no reserve. */
void dion_default_config(dion_config* cfg);

/* Create a context on cfg->device.  Host pointers.  *out is NULL on failure. */
int dion_init(dion_ctx** out, const dion_config* cfg);

/* One Dion step on one matrix (Algorithm 1 + 2).  `a` is a HOST pointer to a
 * descriptor holding DEVICE pointers.  lr is the paper's eta; sqrt(m/n) is
 * applied inside.  If the orthonormalization breaks down, X, M and Q are left
 * unchanged and DION_STATUS_BREAKDOWN is latched.
 *
 * Small matrices (up to 2048 x 2048 elements, r <= 512, fp32 mode on the tensor engine) are launch bound: a
 * step is a chain of ~30 short kernels.  For these the chain is captured into a CUDA graph the first time a
 * descriptor is seen (same pointers, shapes and leading dimensions; the capture runs on a stream of the
 * context, so `cuda_stream` may be the legacy default stream) and later calls with that descriptor replay the
 * graph on `cuda_stream`; lr reaches it through a device scalar, so it may change from call to call.  Up to 64
 * graphs are kept per context (least recently used first out); growing the scratch drops them.  The results
 * are those of the plain launch chain bit for bit.  Steps with per-phase profiling on, grouped, lazy and
 * multi-call steps are always launched plainly. */
int dion_step(dion_ctx* ctx, const dion_matrix* a, float lr, void* cuda_stream);

/* The same step on `count` independent matrices (the paper batches matrices of
 * identical shape; Section 4.1).  Equivalent to `count` dion_step calls in any
 * order, bit for bit.  `list` is a HOST array.  count == 0 is a no-op.
 * Matrices of identical (m, n, r) are stepped together, up to 64 at a time: their
 * large products are launched one after another, the small kernels of the
 * factorization once for all of them.  Each matrix of such a chain needs its own
 * scratch slice, so the context's scratch grows to at most max(16 GiB,
 * dion_config.workspace_bytes), or to one matrix's need if that is larger. */
int dion_step_grouped(dion_ctx* ctx, const dion_matrix* list, int count, float lr, void* cuda_stream);

/* One Lazy-Dion step (Algorithm 6): M <- M + G; if refresh != 0, Q <-
 * Orthonormalize(M^T M Q) (SymPowerIter1); W = M Q; M <- M - (1-mu) W Q^T;
 * X <- X - lr sqrt(m/n) ColNorm(W) Q^T.  colnorm_out receives the norms of W. */
int dion_lazy_step(dion_ctx* ctx, const dion_matrix* a, float lr, int refresh, void* cuda_stream);

/* Scratch bytes a step on (m, n, r) needs; 0 if the shape is invalid. */
size_t dion_workspace_bytes(const dion_ctx* ctx, int64_t m, int64_t n, int64_t r);

/* Compressed data-parallel gradient sync (Section 3.3; the two AllReduce lines of PowerIter1 in
 * Algorithm 2): the step of dion_step in three calls, between which the caller averages the two
 * low-rank factors over the data-parallel ranks (any all-reduce; the library makes no collective
 * call).  Every rank holds the same X and Q, its own gradient G and its own momentum M
 * ("decoupled momentum"); the weight update is the one dion_step makes on the rank-averaged M and
 * G, and the rank average of the M buffers is that step's M.  With one rank and no all-reduce the
 * three calls give dion_step's result.
 *   dion_dp_project: P (m x r, dense, ld = r, DEVICE, 16-byte aligned) <- (M + G) Q; clears *dp_flag.
 *   -- caller: P <- mean over ranks --
 *   dion_dp_factor:  PU holds the averaged P on entry and U = Orthonormalize(P) on return;
 *                    W (n x r, dense, ld = r) <- (M + G)^T U; sets *dp_flag on a breakdown.
 *   -- caller: W <- mean over ranks --
 *   dion_dp_finish:  M <- (M + G) - (1 - mu) U W^T, Q <- ColNorm(W), X <- X - lr sqrt(m/n) U Q^T;
 *                    does nothing (and counts a skipped step) when *dp_flag != 0.
 * `a` must describe the same arrays in the three calls and G must stay unchanged between them;
 * dp_flag is one DEVICE int owned by the caller, one per matrix in flight.  Standard form only;
 * DION_ORTH_RCQR is not available here (DION_ERR_UNSUPPORTED).  Asynchronous on `cuda_stream`. */
int dion_dp_project(dion_ctx* ctx, const dion_matrix* a, float* P, int* dp_flag, void* cuda_stream);
int dion_dp_factor(dion_ctx* ctx, const dion_matrix* a, float* PU, float* W, int* dp_flag, void* cuda_stream);
int dion_dp_finish(dion_ctx* ctx, const dion_matrix* a, const float* U, const float* W, const int* dp_flag,
                   float lr, void* cuda_stream);

/* 1D-sharded Dion (Section 4.1, Algorithm 3): L layers of identical shape, their X, M, G and V sharded by columns
 * over L ranks (rank x holds the columns J_x of every layer and the rows J_x of every V).  The library supplies
 * what a rank computes between the collectives; the caller makes the collectives (any implementation; the
 * library makes no collective call) and the payloads must be in this GPU's memory before a call reads them.
 * `a` describes ONE layer's local shard: m x n_shard arrays X, M, G and Q = V[J_x, :] (n_shard x r; here r may
 * exceed n_shard).  n_total = |J|, the unsharded number of columns (it fixes sqrt(m/n) and the automatic
 * choice of Orthonormalize).  All buffers are DEVICE pointers, dense with leading dimension r, 16-byte aligned.
 *   dion_shard_project (lines 1-2): P (m x r) <- (M + G) V on the shard: this rank's addend of layer l's P;
 *                      clears *flag.
 *   -- caller: ReduceScatter over the ranks along L: rank l receives the sum of every rank's P for layer l --
 *   dion_orthonormalize (line 4, on the rank that owns the layer): PU holds P on entry, U on return;
 *                      sets *flag if the panel broke down.
 *   -- caller: AllGather of U (and of the owners' flags) --
 *   dion_shard_factor  (line 6): W (n_shard x r) <- (M + G)^T U on the shard; colsumsq[r] <- the squared column
 *                      norms of these n_shard rows of W.
 *   -- caller: AllReduce(sum) of colsumsq over the ranks (r numbers per layer) --
 *   dion_shard_finish  (lines 7-10): M <- (M + G) - (1 - mu) U W^T, Q <- W / (sqrt(colsumsq) + eps),
 *                      X <- X - lr sqrt(m / n_total) U Q^T, all on the shard; does nothing (and counts a
 *                      skipped step) when *flag != 0.  colnorm_out, if given, receives sqrt(colsumsq).
 * Every layer's outputs equal those of dion_step on the unsharded layer up to the order of the sums.
 * Standard form only; DION_ORTH_RCQR is not available in dion_orthonormalize.  Asynchronous on `cuda_stream`. */
int dion_shard_project(dion_ctx* ctx, const dion_matrix* a, int64_t n_total, float* P, int* flag, void* cuda_stream);
int dion_orthonormalize(dion_ctx* ctx, int64_t m, int64_t r, int64_t n_total, float* PU, int* flag, void* cuda_stream);
int dion_shard_factor(dion_ctx* ctx, const dion_matrix* a, int64_t n_total, const float* U, float* W, float* colsumsq,
                      const int* flag, void* cuda_stream);
int dion_shard_finish(dion_ctx* ctx, const dion_matrix* a, int64_t n_total, const float* U, const float* W,
                      const float* colsumsq, const int* flag, float lr, void* cuda_stream);

/* Synchronises `cuda_stream`, then reports and clears the latched device status
 * (DION_STATUS_* bits) and the number of steps skipped because of a breakdown
 * since the last call.  Either output pointer may be NULL. */
int dion_get_status(dion_ctx* ctx, void* cuda_stream, int* device_status, int* steps_skipped);

/* Phases of a step, for dion_profile_read. */
enum {
  DION_PHASE_P = 0,       /* P = (M + G) Q                      */
  DION_PHASE_ORTH = 1,    /* U = Orthonormalize(P)              */
  DION_PHASE_R = 2,       /* R = (M + G)^T U                    */
  DION_PHASE_EF = 3,      /* M <- (M + G) - (1 - mu) U R^T      */
  DION_PHASE_COLNORM = 4, /* Q <- ColNorm(R)                    */
  DION_PHASE_X = 5,       /* X <- X - lr sqrt(m/n) U Q^T        */
  DION_PHASE_ORTH_GEMM = 6, /* the part of DION_PHASE_ORTH spent in tensor-core products */
  DION_NUM_PHASES = 7
};

/* Per-phase device timing with CUDA events recorded on the step's own stream.
 * dion_profile_enable(ctx, 1) starts recording (and drops earlier records);
 * dion_profile_enable(ctx, 0) stops.  dion_profile_read synchronises the recorded
 * events, adds up the elapsed milliseconds and the kernel launches of every
 * recorded step per phase into ms[DION_NUM_PHASES] / launches[DION_NUM_PHASES]
 * (host arrays, either may be NULL) and drops the records.  Recording costs two
 * event records per phase; leave it off when not measuring. */
int dion_profile_enable(dion_ctx* ctx, int on);
int dion_profile_read(dion_ctx* ctx, float* ms, int64_t* launches);

/* Synchronises `cuda_stream`, then reports and clears the number of Cholesky QR
 * rounds (the adaptive rounds of DION_ORTH_SHIFTED3, the one or two rounds of
 * DION_ORTH_CHOLQR2) that did work since the last call; rounds skipped on the
 * device are not counted. */
int dion_get_orth_rounds(dion_ctx* ctx, void* cuda_stream, int64_t* rounds);

/* Synchronises `cuda_stream`, then reports and clears the number of matrices whose CholeskyQR2
 * broke down and was redone by the device-side fallback since the last call (the paper reports
 * under 1 % of calls in training). */
int dion_get_fallbacks(dion_ctx* ctx, void* cuda_stream, int64_t* fallbacks);

/* Number of kernel launches issued by this context so far (host counter). */
int64_t dion_launch_count(const dion_ctx* ctx);

/* dion_step for callers that must not allocate device memory.
 *
 * (The paper has no counterpart: this entry point exists for the host program's
 * sake, not for the method's.)
 *
 * Some programs that want to run a Dion step cannot call cudaMalloc at that point:
 * a plug-in running inside another framework's memory pool that has claimed the
 * whole device, a process working under a fixed memory budget negotiated at
 * start-up, or code on a path where the allocator's implicit device-wide
 * synchronisation is not acceptable.  dion_init and dion_step grow their scratch
 * with cudaMalloc; this call never does, and it needs no dion_ctx.  Its scratch
 * (the P/U panels, R, the Gram matrix and its factors, split-K partial sums, the
 * column norms and the step's flags) lives in an array of 24 MiB that is part of
 * the library image, so every GPU that loads the library holds those 24 MiB until
 * the process exits.
 *
 * The step is the one dion_step computes with the default configuration
 * (fp32 products, automatic orthonormalization and engine) and the given mu and
 * eps, on the CURRENT device, asynchronously on `cuda_stream`.  `a` is a HOST
 * pointer; the matrices it names are DEVICE pointers, as for dion_step.
 *
 * Limits and rules:
 *   - A shape whose scratch need exceeds dion_noalloc_scratch_limit() bytes is
 *     rejected with DION_ERR_TOO_LARGE and nothing is launched.  The need is about
 *     4 * (3 * max(m,n) * r + 3 * r * r) bytes plus 10 MiB of fixed buffers; for
 *     example 2048 x 2048 with r = 128 fits, 4096 x 4096 with r = 1024 does not.
 *   - The first call on a device looks up the array's device address and the
 *     device's attributes and has every kernel of the launch chain loaded.  Make
 *     that first call outside any stream capture.  The set-up is guarded by a
 *     mutex, so first calls from several host threads are safe on the host side
 *     (their kernels still share the one array, see the next rule).
 *   - All calls share the one array, which keeps whatever the previous call left
 *     in it; each call clears the words that must start at zero.  Two calls whose
 *     kernels overlap on the GPU (different streams, or several host threads) race
 *     on the array: issue them on one stream, or order them with events.
 *   - A Cholesky breakdown leaves X, M and Q unchanged, as in dion_step, but this
 *     entry point has no status read-out; callers that need one use a dion_ctx.
 *   - It calls no cudaMalloc, cudaFree or other allocating routine. */
int dion_step_noalloc(const dion_matrix* a, float lr, float mu, float eps, void* cuda_stream);

/* Bytes of scratch available to dion_step_noalloc. */
size_t dion_noalloc_scratch_limit(void);

/* Frees the scratch memory and the context.  NULL is allowed. */
void dion_destroy(dion_ctx* ctx);

/* Static string for a DION_ERR_* code. */
const char* dion_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* DION_H_ */

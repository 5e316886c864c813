/*
 * Float64 CPU oracle for the single-device Dion update step.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It exists so that the CUDA
 * library can be checked element by element against a slow, plain and
 * obviously correct restatement of the paper's rule.  Only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it; the CUDA path
 * shares no code, headers, tables or constants with this file.
 *
 * What it follows (paper: "Dion: Distributed Orthonormalized Updates"):
 *   Algorithm 1   X_new = X - eta * O
 *   Algorithm 2   Dion^0D:   B = M + G
 *                            (U, W) = PowerIter1(B, V)
 *                            M_new = B - beta * U W^T        (Eq. 1, error feedback)
 *                            V_new = ColNorm(W)
 *                            O     = sqrt(|I|/|J|) * U V_new^T
 *                 PowerIter1: P = B V ; U = Orthonormalize(P) ; W = B^T U
 *   Section 3.2   Orthonormalize = a standard (Householder) QR
 *   Algorithm 6   Lazy-Dion step between refreshes and SymPowerIter1
 *
 * Notation used here (state names of the library): Q is the paper's V
 * (n x r right factor), R is the paper's W (n x r), mu = 1 - beta.
 *
 * Readings where the paper is silent:
 *   - the QR factor is made unique by requiring diag(R_qr) >= 0;
 *   - ColNorm divides column j by (||column j||_2 + eps), eps passed in;
 *   - the update O uses V_new, the error feedback uses the un-normalised W;
 *   - m = rows = "out" dimension |I|, n = columns = "in" dimension |J|.
 *
 * Parity pins (tests/test_oracle_pins.py): orthonormality of U, the projector
 * form of the error feedback, the full-rank closed form M_new = mu*B, the
 * Frobenius norm of the weight update, two-sided orthogonal equivariance,
 * scale invariance, a rank-1 hand case, a 2x2 hand-worked fixture, static-B
 * subspace iteration against a brute-force SVD, and a cross-check of the
 * Householder factor against a library QR.  Nothing here is "parity unpinned"
 * for full-column-rank P.
 *
 * All matrices are dense, row-major, contiguous, double precision.
 * OpenMP is used only to split independent output rows/columns between host
 * cores; there is no blocking, fusion or re-association of the sums.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef int64_t i64;

int dion_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* C[m x p] = A[m x k] * B[k x p] */
static void mm_nn(i64 m, i64 k, i64 p, const double* A, const double* B, double* C) {
#pragma omp parallel for schedule(static)
  for (i64 i = 0; i < m; ++i) {
    double* c = C + i * p;
    for (i64 j = 0; j < p; ++j) c[j] = 0.0;
    for (i64 l = 0; l < k; ++l) {
      const double a = A[i * k + l];
      const double* b = B + l * p;
      for (i64 j = 0; j < p; ++j) c[j] += a * b[j];
    }
  }
}

/* C[k x p] = A^T * B with A[m x k], B[m x p]: C[j][c] = sum_i A[i][j] B[i][c] */
static void mm_tn(i64 m, i64 k, i64 p, const double* A, const double* B, double* C) {
#pragma omp parallel for schedule(static)
  for (i64 j = 0; j < k; ++j) {
    double* c = C + j * p;
    for (i64 q = 0; q < p; ++q) c[q] = 0.0;
    for (i64 i = 0; i < m; ++i) {
      const double a = A[i * k + j];
      const double* b = B + i * p;
      for (i64 q = 0; q < p; ++q) c[q] += a * b[q];
    }
  }
}

/* C[m x n] -= alpha * A[m x r] * B[n x r]^T */
static void mm_nt_sub(i64 m, i64 n, i64 r, double alpha, const double* A, const double* B, double* C) {
#pragma omp parallel for schedule(static)
  for (i64 i = 0; i < m; ++i) {
    const double* a = A + i * r;
    for (i64 j = 0; j < n; ++j) {
      const double* b = B + j * r;
      double s = 0.0;
      for (i64 l = 0; l < r; ++l) s += a[l] * b[l];
      C[i * n + j] -= alpha * s;
    }
  }
}

/*
 * Thin Householder QR of P (m x r, m >= r), Section 3.2 ("a standard QR").
 * Writes the orthonormal factor to U (m x r) and, if Rqr != NULL, the upper
 * triangular factor (r x r).  Column signs are fixed so that diag(Rqr) >= 0.
 * A column that is already zero below and on the diagonal gets the identity
 * reflector.  Returns the number of such degenerate columns.
 */
int dion_oracle_householder_qr(i64 m, i64 r, const double* P, double* U, double* Rqr) {
  double* A = (double*)malloc(sizeof(double) * (size_t)m * (size_t)r);
  double* V = (double*)calloc((size_t)m * (size_t)r, sizeof(double)); /* reflector j in column j */
  double* w = (double*)malloc(sizeof(double) * (size_t)r);
  int degenerate = 0;
  if (!A || !V || !w) { free(A); free(V); free(w); return -1; }
  memcpy(A, P, sizeof(double) * (size_t)m * (size_t)r);

  for (i64 j = 0; j < r; ++j) {
    double ss = 0.0;
    for (i64 i = j; i < m; ++i) ss += A[i * r + j] * A[i * r + j];
    const double norm = sqrt(ss);
    if (norm == 0.0) { ++degenerate; continue; }          /* H_j = I */
    const double alpha = (A[j * r + j] >= 0.0) ? -norm : norm;
    double vv = 0.0;
    for (i64 i = j; i < m; ++i) {
      double v = A[i * r + j];
      if (i == j) v -= alpha;
      V[i * r + j] = v;
      vv += v * v;
    }
    const double vnorm = sqrt(vv);
    for (i64 i = j; i < m; ++i) V[i * r + j] /= vnorm;
    /* A[j:, j:] -= 2 v (v^T A[j:, j:]) ; columns are independent */
#pragma omp parallel
    {
#ifdef _OPENMP
      const int nt = omp_get_num_threads(), tid = omp_get_thread_num();
#else
      const int nt = 1, tid = 0;
#endif
      const i64 span = r - j;
      const i64 c0 = j + span * tid / nt, c1 = j + span * (tid + 1) / nt;
      if (c1 > c0) {
        for (i64 c = c0; c < c1; ++c) w[c] = 0.0;
        for (i64 i = j; i < m; ++i) {
          const double v = V[i * r + j];
          for (i64 c = c0; c < c1; ++c) w[c] += v * A[i * r + c];
        }
        for (i64 i = j; i < m; ++i) {
          const double v2 = 2.0 * V[i * r + j];
          for (i64 c = c0; c < c1; ++c) A[i * r + c] -= v2 * w[c];
        }
      }
    }
  }

  /* U = H_0 H_1 ... H_{r-1} applied to the first r columns of the identity */
  for (i64 i = 0; i < m; ++i)
    for (i64 c = 0; c < r; ++c) U[i * r + c] = (i == c) ? 1.0 : 0.0;
  for (i64 j = r - 1; j >= 0; --j) {
#pragma omp parallel
    {
#ifdef _OPENMP
      const int nt = omp_get_num_threads(), tid = omp_get_thread_num();
#else
      const int nt = 1, tid = 0;
#endif
      const i64 c0 = r * tid / nt, c1 = r * (tid + 1) / nt;
      if (c1 > c0) {
        for (i64 c = c0; c < c1; ++c) w[c] = 0.0;
        for (i64 i = j; i < m; ++i) {
          const double v = V[i * r + j];
          for (i64 c = c0; c < c1; ++c) w[c] += v * U[i * r + c];
        }
        for (i64 i = j; i < m; ++i) {
          const double v2 = 2.0 * V[i * r + j];
          for (i64 c = c0; c < c1; ++c) U[i * r + c] -= v2 * w[c];
        }
      }
    }
  }

  /* sign convention: diag(R_qr) >= 0 */
  for (i64 j = 0; j < r; ++j) {
    if (A[j * r + j] < 0.0) {
      for (i64 i = 0; i < m; ++i) U[i * r + j] = -U[i * r + j];
      for (i64 c = j; c < r; ++c) A[j * r + c] = -A[j * r + c];
    }
  }
  if (Rqr) {
    for (i64 i = 0; i < r; ++i)
      for (i64 c = 0; c < r; ++c) Rqr[i * r + c] = (c >= i) ? A[i * r + c] : 0.0;
  }
  free(A); free(V); free(w);
  return degenerate;
}

/* ColNorm (Algorithm 2): d_j = ||W[:, j]||_2 ; W[:, j] /= (d_j + eps). */
void dion_oracle_colnorm(i64 n, i64 r, double* W, double eps, double* d) {
  for (i64 j = 0; j < r; ++j) {
    double ss = 0.0;
    for (i64 i = 0; i < n; ++i) ss += W[i * r + j] * W[i * r + j];
    const double dj = sqrt(ss);
    if (d) d[j] = dj;
    for (i64 i = 0; i < n; ++i) W[i * r + j] /= (dj + eps);
  }
}

/*
 * One Dion step (Algorithm 1 + Algorithm 2, unsharded, no DP sync).
 * In place: X, M, Q are overwritten with X_new, M_new, V_new.
 * Optional outputs (may be NULL): d (r column norms of W), P_out (m x r,
 * P = B V before orthonormalization), U_out (m x r), R_out (n x r, W).
 * Returns 0, or -1 if out of host memory, or the number (>0) of degenerate
 * Householder columns (rank-deficient P; outputs then are not unique).
 */
int dion_oracle_step(i64 m, i64 n, i64 r, double* X, double* M, const double* G, double* Q,
                     double mu, double eta, double eps,
                     double* d, double* P_out, double* U_out, double* R_out) {
  double* P = (double*)malloc(sizeof(double) * (size_t)m * (size_t)r);
  double* U = (double*)malloc(sizeof(double) * (size_t)m * (size_t)r);
  double* W = (double*)malloc(sizeof(double) * (size_t)n * (size_t)r);
  if (!P || !U || !W) { free(P); free(U); free(W); return -1; }

  /* Alg. 2 line 1: M <- M + G */
#pragma omp parallel for schedule(static)
  for (i64 i = 0; i < m * n; ++i) M[i] += G[i];
  /* PowerIter1 line 1: P = M V */
  mm_nn(m, n, r, M, Q, P);
  if (P_out) memcpy(P_out, P, sizeof(double) * (size_t)m * (size_t)r);
  /* PowerIter1 line 3: U = Orthonormalize(P) */
  const int degenerate = dion_oracle_householder_qr(m, r, P, U, NULL);
  if (degenerate < 0) { free(P); free(U); free(W); return -1; }
  /* PowerIter1 line 4: W = M^T U */
  mm_tn(m, n, r, M, U, W);
  if (R_out) memcpy(R_out, W, sizeof(double) * (size_t)n * (size_t)r);
  /* Alg. 2 line 3: M_new = M - beta U W^T, beta = 1 - mu */
  mm_nt_sub(m, n, r, 1.0 - mu, U, W, M);
  /* Alg. 2 line 4: V_new = ColNorm(W) */
  dion_oracle_colnorm(n, r, W, eps, d);
  memcpy(Q, W, sizeof(double) * (size_t)n * (size_t)r);
  /* Alg. 2 lines 5-6 and Alg. 1 line 3: X_new = X - eta sqrt(m/n) U V_new^T */
  mm_nt_sub(m, n, r, eta * sqrt((double)m / (double)n), U, Q, X);
  if (U_out) memcpy(U_out, U, sizeof(double) * (size_t)m * (size_t)r);
  free(P); free(U); free(W);
  return degenerate;
}

/*
 * SymPowerIter1 (Algorithm 6): V <- Orthonormalize(M^T M V), in place on Q.
 */
int dion_oracle_sym_power_iter(i64 m, i64 n, i64 r, const double* M, double* Q) {
  double* T = (double*)malloc(sizeof(double) * (size_t)m * (size_t)r);
  double* Z = (double*)malloc(sizeof(double) * (size_t)n * (size_t)r);
  if (!T || !Z) { free(T); free(Z); return -1; }
  mm_nn(m, n, r, M, Q, T);        /* M V        */
  mm_tn(m, n, r, M, T, Z);        /* M^T (M V)  */
  const int degenerate = dion_oracle_householder_qr(n, r, Z, Q, NULL);
  free(T); free(Z);
  return degenerate;
}

/*
 * One Lazy-Dion step (Algorithm 6): M <- M + G; if refresh != 0,
 * V <- SymPowerIter1(M, V); W = M V; M <- M - beta W V^T; U = ColNorm(W);
 * X <- X - eta sqrt(m/n) U V^T.  In place on X, M, Q.  d (optional) receives
 * the r column norms of W.
 */
int dion_oracle_lazy_step(i64 m, i64 n, i64 r, double* X, double* M, const double* G, double* Q,
                          double mu, double eta, double eps, int refresh, double* d) {
  double* W = (double*)malloc(sizeof(double) * (size_t)m * (size_t)r);
  int degenerate = 0;
  if (!W) return -1;
#pragma omp parallel for schedule(static)
  for (i64 i = 0; i < m * n; ++i) M[i] += G[i];
  if (refresh) {
    degenerate = dion_oracle_sym_power_iter(m, n, r, M, Q);
    if (degenerate < 0) { free(W); return -1; }
  }
  mm_nn(m, n, r, M, Q, W);
  mm_nt_sub(m, n, r, 1.0 - mu, W, Q, M);
  dion_oracle_colnorm(m, r, W, eps, d);
  mm_nt_sub(m, n, r, eta * sqrt((double)m / (double)n), W, Q, X);
  free(W);
  return degenerate;
}

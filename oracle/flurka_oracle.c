/*
 * FLuRKA attention forward -- plain fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file defines what the CUDA library must
 * compute; it is slow on purpose, shares no code with the CUDA path and must
 * never be called from it.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg use it.
 *
 * What it follows (arxiv 2306.15799):
 *   Section 3, Eq. (2)   Head = phi(Q) ( phi(E1 K)^T (E2 V) )  -- the optimised
 *                        unification: contract K and V along the sequence
 *                        first, then apply the kernel feature map, then take
 *                        the product in the associative (linear-cost) order.
 *                        The per-head linear maps W^Q, W^K, W^V are taken as
 *                        already applied to the inputs (legal by
 *                        associativity, (E1 K) W^K = E1 (K W^K)), except in
 *                        flurka_oracle_fused_head, which writes them out.
 *   Section 2.1          E1, E2 are d_k x N (here: E, F of shape k x N).
 *                        Kernel attention phi(Q)(phi(K)^T V); random-feature
 *                        maps phi(x) = m^{-1/2} [psi_1(x) .. psi_m(x)] with
 *                        E[psi_i(x) psi_i(y)] = exp(x.y); non-random maps such
 *                        as the exponential linear unit.
 *   Appendix D           the attention weights a kernel method materialises are
 *                        a_nj = phi(x_n).phi(y_j) / sum_j' phi(x_n).phi(y_j'),
 *                        i.e. rows are normalised; Eq. (2) elides this.
 *
 * Readings where the paper is silent:
 *   - positive random features psi_i(x) = exp(w_i.x - |x|^2/2) (FAVOR+);
 *   - the non-random map is phi(x) = elu(x) + 1, alpha = 1, feature dim = d;
 *   - the normaliser sums over the k projected keys;
 *   - no softmax scale is applied here (callers pre-scale Q and K);
 *   - no epsilon is added to the features; non-causal.
 *
 * Stabilisers.  exp(-|k'|^2/2) underflows even fp64 at the benchmark sizes, so
 * with stabilise != 0 the key side subtracts ONE scalar per head (the maximum
 * exponent over all keys and features) and the query side one scalar per row.
 * Both cancel exactly in the ratio.  With stabilise == 0 the formulas are
 * evaluated literally (tiny, well-scaled inputs only).
 *
 * Pins: tests/test_oracle_pins.py checks every function here against closed
 * forms, invariants, brute force and the softmax limit.  The full-size
 * benchmark configurations have no pin beyond the convexity invariant.
 *
 * All arrays are row-major doubles.  Return value 0 = ok, negative = bad
 * argument.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#define FLURKA_ORACLE_PERFORMER 0
#define FLURKA_ORACLE_RNN 1

/* Section 2.1 / Eq. (2): Xp = P X, P is k x N, X is N x d (sequence contraction). */
static void down_project(const double *P, const double *X, int N, int d, int k,
                         double *Xp) {
#pragma omp parallel for schedule(static)
  for (int j = 0; j < k; ++j) {
    double *row = Xp + (size_t)j * d;
    for (int c = 0; c < d; ++c) row[c] = 0.0;
    for (int n = 0; n < N; ++n) {
      const double p = P[(size_t)j * N + n];
      const double *x = X + (size_t)n * d;
      for (int c = 0; c < d; ++c) row[c] += p * x[c];
    }
  }
}

/* Section 2.1: the exponential-linear-unit map, phi(x)_c = elu(x_c) + 1. */
static double elu_plus_one(double x) { return x > 0.0 ? x + 1.0 : exp(x); }

/* Exponent of the positive random feature psi_i(x) = exp(w_i.x - |x|^2 / 2). */
static double feature_exponent(const double *w, const double *x, int d) {
  double dot = 0.0, sq = 0.0;
  for (int c = 0; c < d; ++c) {
    dot += w[c] * x[c];
    sq += x[c] * x[c];
  }
  return dot - 0.5 * sq;
}

/*
 * Feature map of a set of row vectors X (rows x d) -> Phi (rows x p), with
 * p = m for PERFORMER and p = d for RNN.  `scope_global` chooses the
 * stabiliser: one scalar for the whole matrix (key side) or one per row (query
 * side); stabilise == 0 subtracts nothing.  The 1/sqrt(m) of the random-feature
 * map is applied as written in Section 2.1 (it cancels in the ratio).
 */
static void feature_map(const double *X, int rows, int d, const double *W, int m,
                        int variant, int stabilise, int scope_global, double *Phi) {
  if (variant == FLURKA_ORACLE_RNN) {
#pragma omp parallel for schedule(static)
    for (int r = 0; r < rows; ++r)
      for (int c = 0; c < d; ++c)
        Phi[(size_t)r * d + c] = elu_plus_one(X[(size_t)r * d + c]);
    return;
  }
  /* exponents first */
#pragma omp parallel for schedule(static)
  for (int r = 0; r < rows; ++r)
    for (int i = 0; i < m; ++i)
      Phi[(size_t)r * m + i] =
          feature_exponent(W + (size_t)i * d, X + (size_t)r * d, d);
  double gmax = 0.0;
  if (stabilise && scope_global) {
    gmax = -INFINITY;
    for (size_t t = 0; t < (size_t)rows * m; ++t)
      if (Phi[t] > gmax) gmax = Phi[t];
  }
  const double inv_sqrt_m = 1.0 / sqrt((double)m);
#pragma omp parallel for schedule(static)
  for (int r = 0; r < rows; ++r) {
    double s = gmax;
    if (stabilise && !scope_global) {
      s = -INFINITY;
      for (int i = 0; i < m; ++i)
        if (Phi[(size_t)r * m + i] > s) s = Phi[(size_t)r * m + i];
    }
    for (int i = 0; i < m; ++i)
      Phi[(size_t)r * m + i] = exp(Phi[(size_t)r * m + i] - s) * inv_sqrt_m;
  }
}

static int check_args(const void *Q, const void *K, const void *V, const void *E,
                      const void *F, const void *W, int variant, int N, int d,
                      int k, int m, const void *out) {
  if (!Q || !K || !V || !E || !F || !out) return -1;
  if (variant != FLURKA_ORACLE_PERFORMER && variant != FLURKA_ORACLE_RNN) return -2;
  if (variant == FLURKA_ORACLE_PERFORMER && (!W || m <= 0)) return -1;
  if (N <= 0 || d <= 0 || k <= 0) return -3;
  return 0;
}

/* Copies the selected query rows (rows == NULL: all N) into a dense block. */
static double *gather_rows(const double *Q, int d, const long *rows, long n_rows) {
  double *Qs = (double *)malloc((size_t)n_rows * d * sizeof(double));
  if (!Qs) return NULL;
  for (long r = 0; r < n_rows; ++r) {
    const long src = rows ? rows[r] : r;
    memcpy(Qs + (size_t)r * d, Q + (size_t)src * d, (size_t)d * sizeof(double));
  }
  return Qs;
}

/*
 * One head, associative order (Section 2.1 "multiplying out the matrices in an
 * optimal manner"; Appendix B's step list):
 *   1. K' = E K, V' = F V
 *   2. Phi_k = phi(K'), Phi_q = phi(Q)
 *   3. KV = Phi_k^T V'  (p x d),  z = Phi_k^T 1_k  (p)
 *   4. O_n = (Phi_q[n] . KV) / (Phi_q[n] . z)
 * rows/n_rows select query rows (NULL: all).  Optional outputs (may be NULL):
 *   Kp_out, Vp_out [k,d]; KV_out [p,d]; z_out [p]  (as stabilised).
 */
int flurka_oracle_head(const double *Q, const double *K, const double *V,
                       const double *E, const double *F, const double *W,
                       int variant, int N, int d, int k, int m, int stabilise,
                       const long *rows, long n_rows, double *out, double *Kp_out,
                       double *Vp_out, double *KV_out, double *z_out) {
  int rc = check_args(Q, K, V, E, F, W, variant, N, d, k, m, out);
  if (rc) return rc;
  if (!rows) n_rows = N;
  if (n_rows < 0) return -3;
  const int p = (variant == FLURKA_ORACLE_PERFORMER) ? m : d;

  double *Kp = (double *)malloc((size_t)k * d * sizeof(double));
  double *Vp = (double *)malloc((size_t)k * d * sizeof(double));
  double *Phik = (double *)malloc((size_t)k * p * sizeof(double));
  double *KV = (double *)calloc((size_t)p * d, sizeof(double));
  double *z = (double *)calloc((size_t)p, sizeof(double));
  double *Qs = gather_rows(Q, d, rows, n_rows > 0 ? n_rows : 1);
  double *Phiq = (double *)malloc((size_t)(n_rows > 0 ? n_rows : 1) * p * sizeof(double));
  if (!Kp || !Vp || !Phik || !KV || !z || !Qs || !Phiq) {
    free(Kp); free(Vp); free(Phik); free(KV); free(z); free(Qs); free(Phiq);
    return -7;
  }

  /* step 1 */
  down_project(E, K, N, d, k, Kp);
  down_project(F, V, N, d, k, Vp);
  /* step 2 */
  feature_map(Kp, k, d, W, m, variant, stabilise, /*scope_global=*/1, Phik);
  feature_map(Qs, (int)n_rows, d, W, m, variant, stabilise, /*scope_global=*/0, Phiq);
  /* step 3 */
  for (int j = 0; j < k; ++j)
    for (int i = 0; i < p; ++i) {
      const double f = Phik[(size_t)j * p + i];
      z[i] += f;
      for (int c = 0; c < d; ++c) KV[(size_t)i * d + c] += f * Vp[(size_t)j * d + c];
    }
  /* step 4 */
#pragma omp parallel for schedule(static)
  for (long r = 0; r < n_rows; ++r) {
    double den = 0.0;
    double *o = out + (size_t)r * d;
    for (int c = 0; c < d; ++c) o[c] = 0.0;
    for (int i = 0; i < p; ++i) {
      const double f = Phiq[(size_t)r * p + i];
      den += f * z[i];
      for (int c = 0; c < d; ++c) o[c] += f * KV[(size_t)i * d + c];
    }
    for (int c = 0; c < d; ++c) o[c] /= den;
  }

  if (Kp_out) memcpy(Kp_out, Kp, (size_t)k * d * sizeof(double));
  if (Vp_out) memcpy(Vp_out, Vp, (size_t)k * d * sizeof(double));
  if (KV_out) memcpy(KV_out, KV, (size_t)p * d * sizeof(double));
  if (z_out) memcpy(z_out, z, (size_t)p * sizeof(double));
  free(Kp); free(Vp); free(Phik); free(KV); free(z); free(Qs); free(Phiq);
  return 0;
}

/*
 * One head, explicit quadratic form -- the definition of the result
 * (Appendix D's normalised weights applied to Eq. (2)):
 *   A_nj = phi(q_n) . phi(k'_j),  Ahat_nj = A_nj / sum_j' A_nj',  O = Ahat V'.
 * Ahat_out (n_rows x k) is optional.
 */
int flurka_oracle_head_quadratic(const double *Q, const double *K, const double *V,
                                 const double *E, const double *F, const double *W,
                                 int variant, int N, int d, int k, int m,
                                 int stabilise, const long *rows, long n_rows,
                                 double *out, double *Ahat_out) {
  int rc = check_args(Q, K, V, E, F, W, variant, N, d, k, m, out);
  if (rc) return rc;
  if (!rows) n_rows = N;
  if (n_rows < 0) return -3;
  const int p = (variant == FLURKA_ORACLE_PERFORMER) ? m : d;

  double *Kp = (double *)malloc((size_t)k * d * sizeof(double));
  double *Vp = (double *)malloc((size_t)k * d * sizeof(double));
  double *Phik = (double *)malloc((size_t)k * p * sizeof(double));
  double *Qs = gather_rows(Q, d, rows, n_rows > 0 ? n_rows : 1);
  double *Phiq = (double *)malloc((size_t)(n_rows > 0 ? n_rows : 1) * p * sizeof(double));
  if (!Kp || !Vp || !Phik || !Qs || !Phiq) {
    free(Kp); free(Vp); free(Phik); free(Qs); free(Phiq);
    return -7;
  }
  down_project(E, K, N, d, k, Kp);
  down_project(F, V, N, d, k, Vp);
  feature_map(Kp, k, d, W, m, variant, stabilise, 1, Phik);
  feature_map(Qs, (int)n_rows, d, W, m, variant, stabilise, 0, Phiq);

  int fail = 0;
#pragma omp parallel for schedule(static)
  for (long r = 0; r < n_rows; ++r) {
    double *a = (double *)malloc((size_t)k * sizeof(double));
    if (!a) { fail = 1; continue; }
    double rowsum = 0.0;
    for (int j = 0; j < k; ++j) {
      double s = 0.0;
      for (int i = 0; i < p; ++i) s += Phiq[(size_t)r * p + i] * Phik[(size_t)j * p + i];
      a[j] = s;
      rowsum += s;
    }
    double *o = out + (size_t)r * d;
    for (int c = 0; c < d; ++c) o[c] = 0.0;
    for (int j = 0; j < k; ++j) {
      a[j] /= rowsum;
      for (int c = 0; c < d; ++c) o[c] += a[j] * Vp[(size_t)j * d + c];
      if (Ahat_out) Ahat_out[(size_t)r * k + j] = a[j];
    }
    free(a);
  }
  free(Kp); free(Vp); free(Phik); free(Qs); free(Phiq);
  return fail ? -7 : 0;
}

/* Section 2.1 / Appendix B "Linear Transformations": Y = X Wm, X is rows x dm, Wm is dm x d. */
static void linear_map(const double *X, int rows, int dm, const double *Wm, int d, double *Y) {
#pragma omp parallel for schedule(static)
  for (int r = 0; r < rows; ++r) {
    double *y = Y + (size_t)r * d;
    for (int c = 0; c < d; ++c) y[c] = 0.0;
    for (int e = 0; e < dm; ++e) {
      const double x = X[(size_t)r * dm + e];
      const double *w = Wm + (size_t)e * d;
      for (int c = 0; c < d; ++c) y[c] += x * w[c];
    }
  }
}

/*
 * One head of Eq. (2) with its linear maps written out,
 *     Head = phi(Xq W^Q) ( phi((E Xk) W^K)^T ((F Xv) W^V) ),   rows normalised as in Appendix D,
 * in the order the equation and Appendix B's step list give: the un-projected keys and values
 * (N x dm) are contracted along the sequence FIRST (k x dm), the per-head maps (dm x d) are
 * applied to the k contracted rows, the queries are mapped as they are.  Then steps 2 to 4 of
 * flurka_oracle_head.  Xq, Xk, Xv: [N,dm] (they may be the same array); Wq, Wk, Wv: [dm,d], this
 * head's maps; rows / n_rows select query rows (NULL: all).  Optional outputs (may be NULL):
 * Kp_out, Vp_out [k,d] = (E Xk) W^K and (F Xv) W^V; Q_out [n_rows,d] = Xq W^Q.
 */
int flurka_oracle_fused_head(const double *Xq, const double *Xk, const double *Xv,
                             const double *E, const double *F, const double *Wq,
                             const double *Wk, const double *Wv, const double *W, int variant,
                             int N, int dm, int d, int k, int m, int stabilise,
                             const long *rows, long n_rows, double *out, double *Kp_out,
                             double *Vp_out, double *Q_out) {
  int rc = check_args(Xq, Xk, Xv, E, F, W, variant, N, d, k, m, out);
  if (rc) return rc;
  if (!Wq || !Wk || !Wv) return -1;
  if (dm <= 0) return -3;
  if (!rows) n_rows = N;
  if (n_rows < 0) return -3;
  const int p = (variant == FLURKA_ORACLE_PERFORMER) ? m : d;
  const long nq = n_rows > 0 ? n_rows : 1;

  double *Kt = (double *)malloc((size_t)k * dm * sizeof(double));
  double *Vt = (double *)malloc((size_t)k * dm * sizeof(double));
  double *Kp = (double *)malloc((size_t)k * d * sizeof(double));
  double *Vp = (double *)malloc((size_t)k * d * sizeof(double));
  double *Phik = (double *)malloc((size_t)k * p * sizeof(double));
  double *KV = (double *)calloc((size_t)p * d, sizeof(double));
  double *z = (double *)calloc((size_t)p, sizeof(double));
  double *Xs = gather_rows(Xq, dm, rows, nq);
  double *Qs = (double *)malloc((size_t)nq * d * sizeof(double));
  double *Phiq = (double *)malloc((size_t)nq * p * sizeof(double));
  if (!Kt || !Vt || !Kp || !Vp || !Phik || !KV || !z || !Xs || !Qs || !Phiq) {
    free(Kt); free(Vt); free(Kp); free(Vp); free(Phik); free(KV); free(z); free(Xs); free(Qs); free(Phiq);
    return -7;
  }

  /* the low-rank contraction comes before the linear maps */
  down_project(E, Xk, N, dm, k, Kt);
  down_project(F, Xv, N, dm, k, Vt);
  linear_map(Kt, k, dm, Wk, d, Kp);
  linear_map(Vt, k, dm, Wv, d, Vp);
  linear_map(Xs, (int)n_rows, dm, Wq, d, Qs);
  /* feature maps, key-side summaries, ratio: as in flurka_oracle_head */
  feature_map(Kp, k, d, W, m, variant, stabilise, /*one scalar per head*/ 1, Phik);
  feature_map(Qs, (int)n_rows, d, W, m, variant, stabilise, /*one scalar per row*/ 0, Phiq);
  for (int j = 0; j < k; ++j)
    for (int i = 0; i < p; ++i) {
      const double f = Phik[(size_t)j * p + i];
      z[i] += f;
      for (int c = 0; c < d; ++c) KV[(size_t)i * d + c] += f * Vp[(size_t)j * d + c];
    }
#pragma omp parallel for schedule(static)
  for (long r = 0; r < n_rows; ++r) {
    double den = 0.0;
    double *o = out + (size_t)r * d;
    for (int c = 0; c < d; ++c) o[c] = 0.0;
    for (int i = 0; i < p; ++i) {
      const double f = Phiq[(size_t)r * p + i];
      den += f * z[i];
      for (int c = 0; c < d; ++c) o[c] += f * KV[(size_t)i * d + c];
    }
    for (int c = 0; c < d; ++c) o[c] /= den;
  }

  if (Kp_out) memcpy(Kp_out, Kp, (size_t)k * d * sizeof(double));
  if (Vp_out) memcpy(Vp_out, Vp, (size_t)k * d * sizeof(double));
  if (Q_out) memcpy(Q_out, Qs, (size_t)n_rows * d * sizeof(double));
  free(Kt); free(Vt); free(Kp); free(Vp); free(Phik); free(KV); free(z); free(Xs); free(Qs); free(Phiq);
  return 0;
}

/*
 * The feature map on its own (Section 2.1): X is rows x d, Phi is rows x p with
 * p = m (PERFORMER, phi(x) = m^{-1/2} [psi_1(x) .. psi_m(x)]) or p = d (RNN).
 * stabilise / scope_global as in the functions above.
 */
int flurka_oracle_features(const double *X, int rows, int d, const double *W, int m,
                           int variant, int stabilise, int scope_global, double *Phi) {
  if (!X || !Phi || rows <= 0 || d <= 0) return -1;
  if (variant != FLURKA_ORACLE_PERFORMER && variant != FLURKA_ORACLE_RNN) return -2;
  if (variant == FLURKA_ORACLE_PERFORMER && (!W || m <= 0)) return -1;
  feature_map(X, rows, d, W, m, variant, stabilise, scope_global, Phi);
  return 0;
}

/*
 * All heads, associative order.  Q, K, V, out: [B,H,N,d]; E, F: [k,N] shared by
 * every batch and head; W: [m,d] shared (ignored for RNN).
 */
int flurka_oracle_forward(const double *Q, const double *K, const double *V,
                          const double *E, const double *F, const double *W,
                          int variant, int B, int H, int N, int d, int k, int m,
                          double *out) {
  if (B <= 0 || H <= 0) return -3;
  const size_t head = (size_t)N * d;
  for (int bh = 0; bh < B * H; ++bh) {
    int rc = flurka_oracle_head(Q + bh * head, K + bh * head, V + bh * head, E, F, W,
                                variant, N, d, k, m, /*stabilise=*/1, NULL, N,
                                out + bh * head, NULL, NULL, NULL, NULL);
    if (rc) return rc;
  }
  return 0;
}

/* Number of OpenMP threads the loops above will use (1 without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int flurka_oracle_threads(void) { return omp_get_max_threads(); }
#else
int flurka_oracle_threads(void) { return 1; }
#endif

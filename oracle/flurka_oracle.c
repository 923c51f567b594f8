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

/* Derivative of the feature map (Section 2.1) with respect to its argument, contracted with dPhi:
 *   PERFORMER  Phi_i = exp(w_i.x - |x|^2/2 - s)/sqrt(m):  dPhi_i/dx = Phi_i (w_i - x)   (s is a constant
 *              that cancels in the output, so it carries no gradient)
 *   RNN        Phi_c = elu(x_c) + 1:                       dPhi_c/dx_c = 1 for x_c > 0, exp(x_c) otherwise
 * X, dX: rows x d; Phi, dPhi: rows x p.  dX is overwritten. */
static void feature_map_backward(const double *X, int rows, int d, const double *W, int m, int variant,
                                 const double *Phi, const double *dPhi, double *dX) {
#pragma omp parallel for schedule(static)
  for (int r = 0; r < rows; ++r) {
    const double *x = X + (size_t)r * d;
    double *dx = dX + (size_t)r * d;
    if (variant == FLURKA_ORACLE_RNN) {
      for (int c = 0; c < d; ++c)
        dx[c] = dPhi[(size_t)r * d + c] * (x[c] > 0.0 ? 1.0 : exp(x[c]));
      continue;
    }
    for (int c = 0; c < d; ++c) dx[c] = 0.0;
    for (int i = 0; i < m; ++i) {
      const double g = dPhi[(size_t)r * m + i] * Phi[(size_t)r * m + i];
      const double *w = W + (size_t)i * d;
      for (int c = 0; c < d; ++c) dx[c] += g * (w[c] - x[c]);
    }
  }
}

/*
 * Backward pass of one head (the paper trains these models, Sections 1 and 4; it prints no backward
 * formulas, so this is the chain rule applied to steps 1 to 4 of flurka_oracle_head, in reverse):
 * given dO (N x d), the gradients of  sum(O * dO)  with respect to Q, K, V (N x d) and E, F (k x N).
 *   4'. O_n = num_n / den_n:   dnum_n = dO_n / den_n,   dden_n = -(O_n . dO_n) / den_n
 *       num_n = Phi_q[n] KV, den_n = Phi_q[n] . z:
 *       dPhi_q[n,i] = KV_i . dnum_n + z_i dden_n,  dKV_i += Phi_q[n,i] dnum_n,  dz_i += Phi_q[n,i] dden_n
 *   3'. KV = Phi_k^T V', z = Phi_k^T 1:  dPhi_k[j,i] = dKV_i . V'_j + dz_i,  dV'_j = sum_i Phi_k[j,i] dKV_i
 *   2'. through the feature maps (feature_map_backward): dQ, dK'
 *   1'. K' = E K, V' = F V:  dK = E^T dK',  dE = dK' K^T,  dV = F^T dV',  dF = dV' V^T
 * Any of the five outputs may be NULL.
 */
int flurka_oracle_head_backward(const double *Q, const double *K, const double *V, const double *E,
                                const double *F, const double *W, const double *dO, int variant, int N,
                                int d, int k, int m, double *dQ, double *dK, double *dV, double *dE,
                                double *dF) {
  int rc = check_args(Q, K, V, E, F, W, variant, N, d, k, m, dO);
  if (rc) return rc;
  const int p = (variant == FLURKA_ORACLE_PERFORMER) ? m : d;
  double *Kp = (double *)malloc((size_t)k * d * sizeof(double));
  double *Vp = (double *)malloc((size_t)k * d * sizeof(double));
  double *Phik = (double *)malloc((size_t)k * p * sizeof(double));
  double *Phiq = (double *)malloc((size_t)N * p * sizeof(double));
  double *KV = (double *)calloc((size_t)p * d, sizeof(double));
  double *z = (double *)calloc((size_t)p, sizeof(double));
  double *dPhiq = (double *)malloc((size_t)N * p * sizeof(double));
  double *dPhik = (double *)malloc((size_t)k * p * sizeof(double));
  double *dKV = (double *)calloc((size_t)p * d, sizeof(double));
  double *dz = (double *)calloc((size_t)p, sizeof(double));
  double *dKp = (double *)malloc((size_t)k * d * sizeof(double));
  double *dVp = (double *)calloc((size_t)k * d, sizeof(double));
  double *dQl = (double *)malloc((size_t)N * d * sizeof(double));
  if (!Kp || !Vp || !Phik || !Phiq || !KV || !z || !dPhiq || !dPhik || !dKV || !dz || !dKp || !dVp || !dQl) {
    free(Kp); free(Vp); free(Phik); free(Phiq); free(KV); free(z); free(dPhiq); free(dPhik); free(dKV);
    free(dz); free(dKp); free(dVp); free(dQl);
    return -7;
  }
  /* forward, steps 1 to 3 */
  down_project(E, K, N, d, k, Kp);
  down_project(F, V, N, d, k, Vp);
  feature_map(Kp, k, d, W, m, variant, 1, /*one scalar per head*/ 1, Phik);
  feature_map(Q, N, d, W, m, variant, 1, /*one scalar per row*/ 0, Phiq);
  for (int j = 0; j < k; ++j)
    for (int i = 0; i < p; ++i) {
      const double f = Phik[(size_t)j * p + i];
      z[i] += f;
      for (int c = 0; c < d; ++c) KV[(size_t)i * d + c] += f * Vp[(size_t)j * d + c];
    }
  /* step 4 forward and 4' backward, row by row (the sums into dKV, dz are taken serially) */
  for (int n = 0; n < N; ++n) {
    const double *fq = Phiq + (size_t)n * p;
    const double *go = dO + (size_t)n * d;
    double den = 0.0, odo = 0.0;
    for (int i = 0; i < p; ++i) den += fq[i] * z[i];
    for (int c = 0; c < d; ++c) {
      double num = 0.0;
      for (int i = 0; i < p; ++i) num += fq[i] * KV[(size_t)i * d + c];
      odo += (num / den) * go[c];
    }
    const double dden = -odo / den;
    for (int i = 0; i < p; ++i) {
      double acc = z[i] * dden;
      for (int c = 0; c < d; ++c) {
        const double dnum = go[c] / den;
        acc += KV[(size_t)i * d + c] * dnum;
        dKV[(size_t)i * d + c] += fq[i] * dnum;
      }
      dPhiq[(size_t)n * p + i] = acc;
      dz[i] += fq[i] * dden;
    }
  }
  /* 3' */
  for (int j = 0; j < k; ++j)
    for (int i = 0; i < p; ++i) {
      double acc = dz[i];
      for (int c = 0; c < d; ++c) {
        acc += dKV[(size_t)i * d + c] * Vp[(size_t)j * d + c];
        dVp[(size_t)j * d + c] += Phik[(size_t)j * p + i] * dKV[(size_t)i * d + c];
      }
      dPhik[(size_t)j * p + i] = acc;
    }
  /* 2' */
  feature_map_backward(Q, N, d, W, m, variant, Phiq, dPhiq, dQl);
  feature_map_backward(Kp, k, d, W, m, variant, Phik, dPhik, dKp);
  if (dQ) memcpy(dQ, dQl, (size_t)N * d * sizeof(double));
  /* 1' */
#pragma omp parallel for schedule(static)
  for (int n = 0; n < N; ++n) {
    for (int c = 0; c < d; ++c) {
      double gk = 0.0, gv = 0.0;
      for (int j = 0; j < k; ++j) {
        gk += E[(size_t)j * N + n] * dKp[(size_t)j * d + c];
        gv += F[(size_t)j * N + n] * dVp[(size_t)j * d + c];
      }
      if (dK) dK[(size_t)n * d + c] = gk;
      if (dV) dV[(size_t)n * d + c] = gv;
    }
    for (int j = 0; j < k; ++j) {
      double ge = 0.0, gf = 0.0;
      for (int c = 0; c < d; ++c) {
        ge += dKp[(size_t)j * d + c] * K[(size_t)n * d + c];
        gf += dVp[(size_t)j * d + c] * V[(size_t)n * d + c];
      }
      if (dE) dE[(size_t)j * N + n] = ge;
      if (dF) dF[(size_t)j * N + n] = gf;
    }
  }
  free(Kp); free(Vp); free(Phik); free(Phiq); free(KV); free(z); free(dPhiq); free(dPhik); free(dKV);
  free(dz); free(dKp); free(dVp); free(dQl);
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

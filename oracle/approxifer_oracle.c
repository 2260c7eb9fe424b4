/*
 * ApproxIFER reference oracle  --  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of what the ApproxIFER encoder, decoder and
 * error locator compute (arXiv 2109.09868, Section 3 and Appendix A).  It exists
 * so that the CUDA library can be checked against something written directly
 * from the paper's formulas.  It shares no code, header, table or constant with
 * the CUDA path, and nothing in the product may call it.
 *
 * Conventions (the paper writes [n] = {0..n} and has N+1 workers; here
 * W = N+1 is the number of workers, indices i = 0..W-1; K queries per group,
 * indices j = 0..K-1; G independent groups; payload length D (queries) or
 * C (predictions)):
 *
 *   alpha_j = cos((2j+1) pi / (2K))           Chebyshev points, 1st kind (Section 3, encoding)
 *   beta_i  = cos(i pi / (W-1))               Chebyshev points, 2nd kind (Section 3, Eq. "betas")
 *   encode  Xt_i = sum_j l_j(beta_i) X_j,     l_j(z) = [(-1)^j/(z-alpha_j)] / sum_k (-1)^k/(z-alpha_k)
 *   decode  Yh_j = r(alpha_j),                r(z) = sum_{i in F} s_i/(z-beta_i) Yt_i / sum_{i in F} s_i/(z-beta_i)
 *   locate  Algorithm 2 (per class: linear system with Q_0 = 1, a_i = Q(beta_i),
 *           the E smallest |a_i|; then the E most frequent picks).
 *
 * Readings of the paper taken here (each is also a pin in the tests):
 *   - sign s_i in the decoder: default (-1)^(rank of i inside the ascending list F),
 *     which is Berrut's interpolant on the nodes actually used (Section 3,
 *     "Rational Interpolation Background"); flag bit 0 selects the literal
 *     (-1)^i of the decoding equation.  They agree when F is a run of
 *     consecutive workers.
 *   - a node coincidence alpha_j == beta_i is decided by the integer identity
 *     (2j+1)(W-1) == 2 K i and takes the limit value of the interpolant
 *     (weight row = one-hot), because u "passes through the queries".
 *   - "solve the system" with more equations than unknowns = ordinary least
 *     squares on the raw monomial equations.
 *   - ties in "sort by |a_i|" and in "most frequent" go to the lower worker index.
 *
 * Parity pins: every exported function below is pinned by tests that use
 * closed forms, invariants, exact-rational brute force or an independent
 * least-squares routine.  One thing stays "parity unpinned": the values a_i
 * (and hence the vote) when f is not rational, e.g. after a softmax; there the
 * oracle is only "Algorithm 2 followed step by step".
 *
 * Arithmetic: fp64 everywhere, inputs fp32.  No blocking, fusion or
 * re-association beyond what the formulas state; sums run in ascending index
 * order.  Groups are independent and run under an OpenMP parallel-for.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_PI_L 3.14159265358979323846264338327950288419716939937510L

#define ST_NO_WORKERS 1u
#define ST_FEW_WORKERS 2u
#define ST_LOCATE_UNDERDETERMINED 4u
#define ST_NONFINITE 8u
#define ST_ORACLE_RANK_DEFICIENT 0x100u /* oracle-only diagnostic */

#define MAXW 32

/* ------------------------------------------------------------------ threads */

void oracle_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

int oracle_get_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* -------------------------------------------------------------------- nodes */

/* alpha_j = cos((2j+1) pi / (2K)), j = 0..K-1 (Section 3, encoding).  The first
 * half is evaluated in extended precision and rounded once; the second half is
 * the exact mirror image alpha_{K-1-j} = -alpha_j, and the middle node of an
 * odd K is exactly 0. */
void oracle_alpha(int K, double *alpha) {
  for (int j = 0; j < K; ++j) {
    int jm = K - 1 - j;
    if (j < jm)
      alpha[j] = (double)cosl((long double)(2 * j + 1) * ORACLE_PI_L / (long double)(2 * K));
    else if (j == jm)
      alpha[j] = 0.0;
    else
      alpha[j] = -alpha[jm];
  }
}

/* beta_i = cos(i pi / (W-1)), i = 0..W-1 (Section 3, Eq. "betas"; the paper's N
 * is W-1).  Same mirroring: beta_0 = 1, beta_{W-1} = -1, middle node of an odd
 * W exactly 0.  Requires W >= 2. */
void oracle_beta(int W, double *beta) {
  for (int i = 0; i < W; ++i) {
    int im = W - 1 - i;
    if (i < im)
      beta[i] = (double)cosl((long double)i * ORACLE_PI_L / (long double)(W - 1));
    else if (i == im)
      beta[i] = 0.0;
    else
      beta[i] = -beta[im];
  }
}

/* alpha_j == beta_i  <=>  (2j+1)/(2K) == i/(W-1)  <=>  (2j+1)(W-1) == 2 K i. */
int oracle_coincident(int K, int W, int j, int i) {
  return (2 * j + 1) * (W - 1) == 2 * K * i;
}

/* Berrut's interpolant (Eq. 1-2) through (x_k, f_k), k = 0..n-1, x strictly
 * monotone, evaluated at z.  At a node the limit value f_k is returned. */
double oracle_berrut(int n, const double *x, const double *f, double z) {
  double num = 0.0, den = 0.0, sgn = 1.0;
  for (int k = 0; k < n; ++k)
    if (z == x[k]) return f[k];
  for (int k = 0; k < n; ++k) {
    double t = sgn / (z - x[k]);
    num += t * f[k];
    den += t;
    sgn = -sgn;
  }
  return num / den;
}

/* ------------------------------------------------------------------ encoder */

/* e[i*K + j] = l_j(beta_i) (Section 3, the basis functions of u). */
void oracle_encode_weights(int K, int W, double *e) {
  double alpha[MAXW], beta[MAXW];
  oracle_alpha(K, alpha);
  oracle_beta(W, beta);
  for (int i = 0; i < W; ++i) {
    int hit = -1;
    for (int j = 0; j < K; ++j)
      if (oracle_coincident(K, W, j, i)) hit = j;
    if (hit >= 0) {
      for (int j = 0; j < K; ++j) e[i * K + j] = (j == hit) ? 1.0 : 0.0;
      continue;
    }
    double t[MAXW], den = 0.0, sgn = 1.0;
    for (int j = 0; j < K; ++j) {
      t[j] = sgn / (beta[i] - alpha[j]);
      den += t[j];
      sgn = -sgn;
    }
    for (int j = 0; j < K; ++j) e[i * K + j] = t[j] / den;
  }
}

/* Xt[g][i][:] = u(beta_i) = sum_j l_j(beta_i) X[g][j][:]  (Section 3, encoding).
 * Strides are in elements; the innermost dimension is contiguous. */
void oracle_encode(int K, int W, int64_t G, int64_t D, const float *X, int64_t x_gs, int64_t x_rs,
                   double *Xt, int64_t o_gs, int64_t o_rs) {
  double e[MAXW * MAXW];
  oracle_encode_weights(K, W, e);
#pragma omp parallel for schedule(static)
  for (int64_t g = 0; g < G; ++g) {
    for (int i = 0; i < W; ++i) {
      double *out = Xt + g * o_gs + (int64_t)i * o_rs;
      for (int64_t d = 0; d < D; ++d) out[d] = 0.0;
      for (int j = 0; j < K; ++j) {
        const float *x = X + g * x_gs + (int64_t)j * x_rs;
        double w = e[i * K + j];
        if (w == 0.0) continue; /* one-hot rows copy their query exactly */
        for (int64_t d = 0; d < D; ++d) out[d] += w * (double)x[d];
      }
    }
  }
}

/* ------------------------------------------------------------------ decoder */

/* Ascending list F of the workers i < W whose mask bit is set; returns |F|. */
int oracle_compact(int W, uint32_t mask, int *F) {
  int n = 0;
  for (int i = 0; i < W; ++i)
    if ((mask >> i) & 1u) F[n++] = i;
  return n;
}

/* w[j*W + r], r = 0..n-1: weight of worker F[r] in Yh_j = r(alpha_j)
 * (Section 3, decoding).  flags bit 0: 0 = sign (-1)^r, 1 = sign (-1)^F[r]. */
int oracle_decode_weights(int K, int W, uint32_t flags, uint32_t mask, double *w, int *F) {
  double alpha[MAXW], beta[MAXW];
  oracle_alpha(K, alpha);
  oracle_beta(W, beta);
  int n = oracle_compact(W, mask, F);
  for (int j = 0; j < K; ++j) {
    int hit = -1;
    for (int r = 0; r < n; ++r)
      if (oracle_coincident(K, W, j, F[r])) hit = r;
    if (hit >= 0) {
      for (int r = 0; r < n; ++r) w[j * W + r] = (r == hit) ? 1.0 : 0.0;
      continue;
    }
    double t[MAXW], den = 0.0;
    for (int r = 0; r < n; ++r) {
      int e = (flags & 1u) ? F[r] : r;
      double s = (e & 1) ? -1.0 : 1.0;
      t[r] = s / (alpha[j] - beta[F[r]]);
      den += t[r];
    }
    for (int r = 0; r < n; ++r) w[j * W + r] = t[r] / den;
  }
  return n;
}

/* Yh[g][j][:] = r(alpha_j) over the workers present in mask[g].  Rows of absent
 * workers are never touched.  n_used and status may be NULL. */
void oracle_decode(int K, int W, uint32_t flags, int64_t G, int64_t C, const float *Yt, int64_t y_gs,
                   int64_t y_rs, const uint32_t *mask, double *Yh, int64_t o_gs, int64_t o_rs,
                   int32_t *n_used, uint32_t *status) {
#pragma omp parallel for schedule(static)
  for (int64_t g = 0; g < G; ++g) {
    double w[MAXW * MAXW];
    int F[MAXW];
    int n = oracle_decode_weights(K, W, flags, mask[g], w, F);
    uint32_t st = 0;
    if (n == 0) st |= ST_NO_WORKERS;
    if (n < K) st |= ST_FEW_WORKERS;
    for (int j = 0; j < K; ++j) {
      double *out = Yh + g * o_gs + (int64_t)j * o_rs;
      for (int64_t c = 0; c < C; ++c) out[c] = 0.0;
      for (int r = 0; r < n; ++r) {
        const float *y = Yt + g * y_gs + (int64_t)F[r] * y_rs;
        double wr = w[j * W + r];
        if (wr == 0.0) continue;
        for (int64_t c = 0; c < C; ++c) out[c] += wr * (double)y[c];
      }
    }
    if (n_used) n_used[g] = n;
    if (status) status[g] = st;
  }
}

/* ------------------------------------------------------------------ locator */

/* Least squares min ||A x - b||_2 by Householder QR with column pivoting.
 * A is n x p, column-major (A[r + n*c]), overwritten; b overwritten.
 * Returns the numerical rank; columns beyond the rank get x = 0. */
static int ls_solve(int n, int p, double *A, double *b, double *x) {
  int perm[2 * MAXW];
  double diag0 = 0.0;
  int rank = p;
  for (int c = 0; c < p; ++c) perm[c] = c;
  for (int k = 0; k < p; ++k) {
    /* pivot: remaining column with the largest norm below row k */
    int piv = k;
    double best = -1.0;
    for (int c = k; c < p; ++c) {
      double s = 0.0;
      for (int r = k; r < n; ++r) s += A[r + n * c] * A[r + n * c];
      if (s > best) {
        best = s;
        piv = c;
      }
    }
    if (piv != k) {
      for (int r = 0; r < n; ++r) {
        double t = A[r + n * k];
        A[r + n * k] = A[r + n * piv];
        A[r + n * piv] = t;
      }
      int t = perm[k];
      perm[k] = perm[piv];
      perm[piv] = t;
    }
    double normx = sqrt(best);
    if (k == 0) diag0 = normx;
    if (!(normx > 1e-13 * diag0)) { /* also catches NaN */
      rank = k;
      break;
    }
    /* reflector H = I - 2 v v^T / (v^T v) mapping column k to (akk, 0, ..)^T */
    double akk = (A[k + n * k] >= 0.0) ? -normx : normx;
    double v[MAXW];
    double vv = 0.0;
    for (int r = k; r < n; ++r) v[r] = A[r + n * k];
    v[k] -= akk;
    for (int r = k; r < n; ++r) vv += v[r] * v[r];
    for (int c = k + 1; c < p; ++c) {
      double s = 0.0;
      for (int r = k; r < n; ++r) s += v[r] * A[r + n * c];
      s = 2.0 * s / vv;
      for (int r = k; r < n; ++r) A[r + n * c] -= s * v[r];
    }
    {
      double s = 0.0;
      for (int r = k; r < n; ++r) s += v[r] * b[r];
      s = 2.0 * s / vv;
      for (int r = k; r < n; ++r) b[r] -= s * v[r];
    }
    A[k + n * k] = akk;
    for (int r = k + 1; r < n; ++r) A[r + n * k] = 0.0;
  }
  double z[2 * MAXW];
  for (int k = rank - 1; k >= 0; --k) {
    double s = b[k];
    for (int c = k + 1; c < rank; ++c) s -= A[k + n * c] * z[c];
    z[k] = s / A[k + n * k];
  }
  for (int c = 0; c < p; ++c) x[c] = 0.0;
  for (int k = 0; k < rank; ++k) x[perm[k]] = z[k];
  return rank;
}

/* One pass of Algorithm 2's loop body for a single class (Steps 1-3):
 * nodes xs[r] (the beta of the r-th available worker), values y[r], r < n,
 * m = K+E.  Unknowns x = (P_0..P_{m-1}, Q_1..Q_{m-1}); equations
 *   sum_k P_k xs^k - y sum_{k>=1} Q_k xs^k = y        (Q_0 = 1 moved right)
 * solved in the least-squares sense; a[r] = Q(xs[r]).  Returns the rank. */
int oracle_locate_class(int n, int m, const double *xs, const double *y, double *x, double *a) {
  int p = 2 * m - 1;
  double A[MAXW * 2 * MAXW], b[MAXW];
  for (int r = 0; r < n; ++r) {
    double pw = 1.0;
    for (int k = 0; k < m; ++k) {
      A[r + n * k] = pw;
      if (k >= 1) A[r + n * (m - 1 + k)] = -y[r] * pw;
      pw *= xs[r];
    }
    b[r] = y[r];
  }
  int rank = ls_solve(n, p, A, b, x);
  for (int r = 0; r < n; ++r) {
    double q = 1.0, pw = xs[r];
    for (int k = 1; k < m; ++k) {
      q += x[m - 1 + k] * pw;
      pw *= xs[r];
    }
    a[r] = q;
  }
  return rank;
}

/* Algorithm 2 for G groups.
 *   adv[g][0..E-1]   located workers, ascending (-1 when nothing was located)
 *   trusted[g]       mask[g] (bits < W) with the located workers cleared
 *   status[g]        ST_* bits (may be NULL)
 *   min_gap[g]       min over classes of |a|_(E+1) / |a|_(E)  (>= 1; how far the
 *                    E-th pick is from the runner-up; may be NULL)
 *   vote_margin[g]   votes of the E-th elected worker minus votes of the best
 *                    non-elected one (0 = decided by the tie rule; may be NULL)
 */
void oracle_locate(int K, int W, int E, int64_t G, int64_t C, const float *Yt, int64_t y_gs,
                   int64_t y_rs, const uint32_t *mask, int32_t *adv, uint32_t *trusted,
                   uint32_t *status, double *min_gap, int32_t *vote_margin) {
  double beta[MAXW];
  oracle_beta(W, beta);
  const int m = K + E;
  const uint32_t wmask = (W >= 32) ? 0xffffffffu : ((1u << W) - 1u);
#pragma omp parallel for schedule(dynamic, 16)
  for (int64_t g = 0; g < G; ++g) {
    int F[MAXW];
    uint32_t mk = mask[g] & wmask;
    int n = oracle_compact(W, mk, F);
    uint32_t st = 0;
    double gap = INFINITY;
    int margin = 0;
    if (n < 2 * m || E <= 0) {
      if (E > 0) st |= ST_LOCATE_UNDERDETERMINED;
      for (int e = 0; e < E; ++e) adv[g * E + e] = -1;
      trusted[g] = mk;
    } else {
      int votes[MAXW];
      for (int i = 0; i < W; ++i) votes[i] = 0;
      double xs[MAXW];
      for (int r = 0; r < n; ++r) xs[r] = beta[F[r]];
      for (int64_t c = 0; c < C; ++c) {
        double y[MAXW], x[2 * MAXW], a[MAXW], mag[MAXW];
        for (int r = 0; r < n; ++r) y[r] = (double)Yt[g * y_gs + (int64_t)F[r] * y_rs + c];
        int rank = oracle_locate_class(n, m, xs, y, x, a);
        if (rank < 2 * m - 1) st |= ST_ORACLE_RANK_DEFICIENT;
        for (int r = 0; r < n; ++r) {
          mag[r] = fabs(a[r]);
          if (!isfinite(a[r])) {
            mag[r] = INFINITY;
            st |= ST_NONFINITE;
          }
        }
        /* Steps 4-5: the E smallest |a_i|, ties to the lower worker index */
        int taken[MAXW];
        for (int r = 0; r < n; ++r) taken[r] = 0;
        double last = 0.0;
        for (int e = 0; e <= E && e < n; ++e) {
          int best = -1;
          for (int r = 0; r < n; ++r)
            if (!taken[r] && (best < 0 || mag[r] < mag[best])) best = r;
          taken[best] = 1;
          if (e < E) {
            votes[F[best]] += 1;
            last = mag[best];
          } else {
            double ratio = (last > 0.0) ? mag[best] / last : INFINITY;
            if (ratio < gap) gap = ratio;
          }
        }
      }
      /* the E most frequent workers, ties to the lower index */
      int elected[MAXW];
      for (int i = 0; i < W; ++i) elected[i] = 0;
      int last_votes = 0;
      for (int e = 0; e <= E; ++e) {
        int best = -1;
        for (int i = 0; i < W; ++i)
          if (((mk >> i) & 1u) && !elected[i] && (best < 0 || votes[i] > votes[best])) best = i;
        if (e < E) {
          elected[best] = 1;
          last_votes = votes[best];
        } else {
          margin = last_votes - (best >= 0 ? votes[best] : 0);
        }
      }
      int e = 0;
      uint32_t bits = 0;
      for (int i = 0; i < W; ++i)
        if (elected[i]) {
          adv[g * E + e++] = i;
          bits |= 1u << i;
        }
      trusted[g] = mk & ~bits;
    }
    if (status) status[g] = st;
    if (min_gap) min_gap[g] = gap;
    if (vote_margin) vote_margin[g] = margin;
  }
}

/*
 * Factored Gossip DiLoCo -- float64 CPU oracle of one outer round.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * outer synchronisation round computes, written from the paper's equations.  It
 * shares no code with the CUDA library, is never called by the product path, and
 * is only used by the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * Every array is a C-contiguous [K][P] matrix of doubles: row m = worker m,
 * P = flat parameter count.  Mixing matrices are dense row-major [K][K] doubles
 * in the ROW convention of the paper's definition of Mix_W:
 *     Mix_W(v)_m = sum_n W[m][n] * v_n            (Sec. 3, "Gossip-based Mixing")
 * so row m of W holds the weights worker m applies.  No blocking, no fusion, no
 * reordering: each function is one equation written as loops, and the sums over
 * workers run n = 0..K-1 in that order.
 *
 * The only parallelism is an OpenMP "parallel for" over the independent columns
 * (or rows) of a loop nest; it changes no arithmetic and no summation order.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Number of host threads the loops below will use. */
int fgdo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void fgdo_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/*
 * Outer gradient.  The paper defines the outer pseudo-gradient of worker m as
 * Delta_m = y_{m,r,H} - y_{m,r,0} (Sec. 4 round equations; Algorithm 1, the line
 * computing Delta) and hands the outer optimizer the NEGATED mixed value
 * (OuterOpt(x, -Delta_hat)).  With theta_prev = y_{m,r,0} = z_{m,r} and
 * theta_local = y_{m,r,H} the gradient the optimizer sees before mixing is
 *     g[m][p] = theta_prev[m][p] - theta_local[m][p] = -Delta_m[p].
 */
void fgdo_outer_grad(int K, int64_t P, const double* theta_prev,
                     const double* theta_local, double* g) {
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < P; ++p)
    for (int m = 0; m < K; ++m)
      g[(size_t)m * P + p] = theta_prev[(size_t)m * P + p] - theta_local[(size_t)m * P + p];
}

/*
 * Gossip mixing, the definition in Sec. 3:  out_m = sum_{n} W[m][n] * in_n.
 * Global averaging is the special case W = (1/K) 1 1^T, identity is W = I.
 * in and out must not overlap.
 */
void fgdo_mix(int K, int64_t P, const double* W, const double* in, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < P; ++p)
    for (int m = 0; m < K; ++m) {
      double acc = 0.0;
      for (int n = 0; n < K; ++n) acc += W[m * K + n] * in[(size_t)n * P + p];
      out[(size_t)m * P + p] = acc;
    }
}

/*
 * Outer optimizer: SGD with Nesterov momentum in the form the paper prints in
 * App. B ("Momentum Update" / "Optimization Step"), applied to the Mix1 output
 * x_m and the mixed gradient ghat_m of worker m:
 *     v'[m][p]        = mu * v[m][p] + ghat[m][p]
 *     theta_new[m][p] = x[m][p] - gamma * (ghat[m][p] + mu * v'[m][p])
 * v is updated in place.  theta_new may not overlap x or ghat.
 */
void fgdo_nesterov(int K, int64_t P, const double* x, const double* ghat, double* v,
                   double gamma, double mu, double* theta_new) {
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < P; ++p)
    for (int m = 0; m < K; ++m) {
      size_t i = (size_t)m * P + p;
      double vn = mu * v[i] + ghat[i];
      v[i] = vn;
      theta_new[i] = x[i] - gamma * (ghat[i] + mu * vn);
    }
}

/*
 * One outer round of Factored Gossip DiLoCo for all K workers (Sec. 4 round
 * equations, Algorithm 1), in the paper's order:
 *     x_m      = Mix1(theta_prev)_m                   (non-blocking mix of z_{m,r})
 *     g_m      = theta_prev_m - theta_local_m         (= -Delta_m)
 *     ghat_m   = Mix2(g)_m                            (blocking mix; Mix2 is linear,
 *                                                      so Mix2(-Delta) = -Mix2(Delta))
 *     z_{m,r+1}= OuterOpt(x_m, ghat_m)                (Nesterov SGD, App. B)
 * x_out and ghat_out (each [K][P]) receive the intermediate values when non-NULL.
 * Returns 0, or -1 if scratch memory could not be allocated.
 */
int fgdo_round(int K, int64_t P, const double* W1, const double* W2,
               const double* theta_prev, const double* theta_local, double* v,
               double gamma, double mu, double* theta_new, double* x_out,
               double* ghat_out) {
  size_t n = (size_t)K * (size_t)P;
  double* x = x_out ? x_out : (double*)malloc(n * sizeof(double));
  double* g = (double*)malloc(n * sizeof(double));
  double* ghat = ghat_out ? ghat_out : (double*)malloc(n * sizeof(double));
  int rc = -1;
  if (x && g && ghat) {
    fgdo_mix(K, P, W1, theta_prev, x);
    fgdo_outer_grad(K, P, theta_prev, theta_local, g);
    fgdo_mix(K, P, W2, g, ghat);
    fgdo_nesterov(K, P, x, ghat, v, gamma, mu, theta_new);
    rc = 0;
  }
  if (!x_out) free(x);
  free(g);
  if (!ghat_out) free(ghat);
  return rc;
}

/*
 * Consensus distance ingredients (Sec. 4.4 L2 consensus distance; App. D "L2
 * Parameter Disagreement"):
 *     mean[p] = (1/K) sum_m theta[m][p]
 *     s[m]    = sum_p (theta[m][p] - mean[p])^2
 * Both of the paper's definitions follow from s: the main-text one is
 * (1/K) sum_m sqrt(s[m]), the appendix one is (1/K) sum_m s[m].
 * The sum over p is a compensated (Neumaier) double sum so that the reference
 * is accurate to the last few bits at any P.
 */
int fgdo_consensus_sumsq(int K, int64_t P, const double* theta, double* s) {
  double* mean = (double*)malloc((size_t)P * sizeof(double));
  if (!mean) return -1;
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < P; ++p) {
    double acc = 0.0;
    for (int m = 0; m < K; ++m) acc += theta[(size_t)m * P + p];
    mean[p] = acc / (double)K;
  }
#pragma omp parallel for schedule(static)
  for (int m = 0; m < K; ++m) {
    double sum = 0.0, comp = 0.0;
    for (int64_t p = 0; p < P; ++p) {
      double d = theta[(size_t)m * P + p] - mean[p];
      double t = d * d;
      double u = sum + t;
      if (fabs(sum) >= fabs(t)) comp += (sum - u) + t; else comp += (t - u) + sum;
      sum = u;
    }
    s[m] = sum + comp;
  }
  free(mean);
  return 0;
}

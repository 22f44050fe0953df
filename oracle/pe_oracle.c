/*
 * CPU oracle for per-example gradient statistics of a linear layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
 * method computes; it exists so that the CUDA library can be checked against
 * something written independently from the paper.  It shares no code with the
 * CUDA path and nothing in the product may call it.
 *
 * Conventions: X is [B, T, d_in], dY is [B, T, d_out], both row-major.  Outputs
 * are [d_out, d_in] row-major (the transpose of the paper's D x F layout, same
 * numbers).  All arithmetic is fp64; inputs are either fp32 or bf16 bit patterns
 * and are widened exactly.
 *
 * Every function here follows the "one example at a time" route of Section 2.1
 * (the compute-intensive implementation): form the gradient of example b, apply
 * phi to it, add it to the running sum over b.  That is the definition of the
 * statistic in Eq. (2) with the 1/B left to the caller.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* bf16 -> double: a bf16 is the upper half of an IEEE binary32. */
static double widen_bf16(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* Copy rows [row0, row0+rows) of a [*, width] matrix into doubles. */
static void widen_rows(const void* src, int is_bf16, long long row0, long long rows, long long width,
                       double* dst) {
  long long n = rows * width, off = row0 * width;
  if (is_bf16) {
    const uint16_t* p = (const uint16_t*)src + off;
    for (long long k = 0; k < n; ++k) dst[k] = widen_bf16(p[k]);
  } else {
    const float* p = (const float*)src + off;
    for (long long k = 0; k < n; ++k) dst[k] = (double)p[k];
  }
}

static double sign3(double g) { return (g > 0.0) - (g < 0.0); } /* sign(0) = 0 */

/*
 * Sequence-level per-example statistics (Section 2.3, "Dense layers in
 * sequence-level architectures"): for each example b the gradient is the
 * contraction over that sequence's tokens only,
 *     G_b[o,i] = sum_t dY[b,t,o] * X[b,t,i],
 * phi is applied to the whole G_b (after the sum over t) and the results are
 * summed over b (Eq. (2), Eq. (3), and the sign statistic of Section 3.1).
 *
 *   sum_g   [d_out*d_in]  = sum_b G_b                (the ordinary batch gradient)
 *   sum_g2  [d_out*d_in]  = sum_b G_b^2
 *   sum_sgn [d_out*d_in]  = sum_b sign(G_b),  sign(0) = 0
 *   max_abs [B]           = max_{o,i} |G_b[o,i]|
 *   n_small [d_out*d_in]  = number of examples b with |G_b[o,i]| <= small_rel * max_abs[b]
 *                           (entries whose sign a lower-precision evaluation may flip)
 * Any output pointer may be NULL.  Returns 0, or 1 on bad arguments / allocation failure.
 */
int oracle_linear_stats(const void* X, const void* dY, int is_bf16, int B, int T, int d_in, int d_out,
                        double small_rel, double* sum_g, double* sum_g2, double* sum_sgn,
                        double* max_abs, int32_t* n_small) {
  if (!X || !dY || B < 0 || T < 0 || d_in <= 0 || d_out <= 0) return 1;
  long long n = (long long)d_out * d_in;
  double* G = (double*)malloc(sizeof(double) * (size_t)n);
  double* xb = (double*)malloc(sizeof(double) * (size_t)((long long)(T > 0 ? T : 1) * d_in));
  double* yb = (double*)malloc(sizeof(double) * (size_t)((long long)(T > 0 ? T : 1) * d_out));
  if (!G || !xb || !yb) { free(G); free(xb); free(yb); return 1; }
  for (long long k = 0; k < n; ++k) {
    if (sum_g) sum_g[k] = 0.0;
    if (sum_g2) sum_g2[k] = 0.0;
    if (sum_sgn) sum_sgn[k] = 0.0;
    if (n_small) n_small[k] = 0;
  }
  for (int b = 0; b < B; ++b) {
    widen_rows(X, is_bf16, (long long)b * T, T, d_in, xb);
    widen_rows(dY, is_bf16, (long long)b * T, T, d_out, yb);
    /* G_b = dY_b^T X_b, contracted over this example's T tokens. */
#pragma omp parallel for schedule(static)
    for (int o = 0; o < d_out; ++o) {
      double* g = G + (long long)o * d_in;
      for (int i = 0; i < d_in; ++i) g[i] = 0.0;
      for (int t = 0; t < T; ++t) {
        double lam = yb[(long long)t * d_out + o];
        const double* h = xb + (long long)t * d_in;
        for (int i = 0; i < d_in; ++i) g[i] += lam * h[i];
      }
    }
    double mx = 0.0;
    for (long long k = 0; k < n; ++k) {
      double a = fabs(G[k]);
      if (a > mx) mx = a;
    }
    if (max_abs) max_abs[b] = mx;
    /* phi, then the sum over examples. */
    for (long long k = 0; k < n; ++k) {
      double g = G[k];
      if (sum_g) sum_g[k] += g;
      if (sum_g2) sum_g2[k] += g * g;
      if (sum_sgn) sum_sgn[k] += sign3(g);
      if (n_small && fabs(g) <= small_rel * mx) n_small[k] += 1;
    }
  }
  free(G); free(xb); free(yb);
  return 0;
}

/*
 * Per-example squared gradient norms (Section 2.3: the quantity N_b = ||grad_W f(theta; x_b)||_2^2 of the
 * "ghost clipping" remark; what a clipping phi of Section 2.1 needs):
 *     N_b = sum_{o,i} G_b[o,i]^2,     G_b[o,i] = sum_t dY[b,t,o] * X[b,t,i],
 * computed the long way: the whole G_b is formed, then its entries are squared and summed.
 */
int oracle_example_sqnorms(const void* X, const void* dY, int is_bf16, int B, int T, int d_in, int d_out,
                           double* norms) {
  if (!X || !dY || !norms || B < 0 || T < 0 || d_in <= 0 || d_out <= 0) return 1;
  double* row = (double*)malloc(sizeof(double) * (size_t)d_out);
  double* xb = (double*)malloc(sizeof(double) * (size_t)((long long)(T > 0 ? T : 1) * d_in));
  double* yb = (double*)malloc(sizeof(double) * (size_t)((long long)(T > 0 ? T : 1) * d_out));
  if (!row || !xb || !yb) { free(row); free(xb); free(yb); return 1; }
  for (int b = 0; b < B; ++b) {
    widen_rows(X, is_bf16, (long long)b * T, T, d_in, xb);
    widen_rows(dY, is_bf16, (long long)b * T, T, d_out, yb);
#pragma omp parallel for schedule(static)
    for (int o = 0; o < d_out; ++o) {
      double acc = 0.0;
      for (int i = 0; i < d_in; ++i) {
        double g = 0.0;
        for (int t = 0; t < T; ++t) g += yb[(long long)t * d_out + o] * xb[(long long)t * d_in + i];
        acc += g * g;
      }
      row[o] = acc;
    }
    double nb = 0.0;
    for (int o = 0; o < d_out; ++o) nb += row[o];
    norms[b] = nb;
  }
  free(row); free(xb); free(yb);
  return 0;
}

/*
 * Per-token second moment (Section 2.3, the "per-token" alternative):
 *     S'[o,i] = sum_{b,t} dY[b,t,o]^2 * X[b,t,i]^2 ,
 * one term per (example, token) row; B and T only enter as the row count.
 */
int oracle_token_sqstats(const void* X, const void* dY, int is_bf16, int B, int T, int d_in, int d_out,
                         double* out) {
  if (!X || !dY || !out || B < 0 || T < 0 || d_in <= 0 || d_out <= 0) return 1;
  long long rows = (long long)B * T;
  long long n = (long long)d_out * d_in;
  double* xr = (double*)malloc(sizeof(double) * (size_t)d_in);
  double* yr = (double*)malloc(sizeof(double) * (size_t)d_out);
  if (!xr || !yr) { free(xr); free(yr); return 1; }
  for (long long k = 0; k < n; ++k) out[k] = 0.0;
  for (long long r = 0; r < rows; ++r) {
    widen_rows(X, is_bf16, r, 1, d_in, xr);
    widen_rows(dY, is_bf16, r, 1, d_out, yr);
    for (int i = 0; i < d_in; ++i) xr[i] = xr[i] * xr[i];
#pragma omp parallel for schedule(static)
    for (int o = 0; o < d_out; ++o) {
      double l2 = yr[o] * yr[o];
      double* s = out + (long long)o * d_in;
      for (int i = 0; i < d_in; ++i) s[i] += l2 * xr[i];
    }
  }
  free(xr); free(yr);
  return 0;
}

/*
 * One MicroAdam step (Algorithm 1, MicroAdam branch; Eq. (3) for nu):
 *   mu = s * sum_g / B                       average per-example gradient, g_b = s * G_b
 *   nu = s^2 * sum_g2 / B                    average element-wise square
 *   m  = beta1 m + (1 - beta1) mu
 *   v  = beta2 v + (1 - beta2) nu
 *   mh = m / (1 - beta1^t),  vh = v / (1 - beta2^t)
 *   u  = mh / (sqrt(vh) + eps)               eps_inside_sqrt == 0  (Section 3.2.3's form)
 *   u  = mh / sqrt(eps + vh)                 eps_inside_sqrt != 0  (Algorithm 1 as printed)
 *   theta = theta - lr * u - wd * theta      decay not multiplied by lr (Appendix E)
 * theta, m, v are updated in place.  step is 1-based.
 */
int oracle_microadam_step(double* theta, double* m, double* v, const double* sum_g, const double* sum_g2,
                          long long n, int B, double grad_scale, double lr, double beta1, double beta2,
                          double eps, int eps_inside_sqrt, double weight_decay, int step) {
  if (!theta || !m || !v || !sum_g || !sum_g2 || n < 0 || B < 1 || step < 1) return 1;
  double c1 = 1.0 - pow(beta1, (double)step);
  double c2 = 1.0 - pow(beta2, (double)step);
  for (long long k = 0; k < n; ++k) {
    double mu = grad_scale * sum_g[k] / (double)B;
    double nu = grad_scale * grad_scale * sum_g2[k] / (double)B;
    m[k] = beta1 * m[k] + (1.0 - beta1) * mu;
    v[k] = beta2 * v[k] + (1.0 - beta2) * nu;
    double mh = m[k] / c1;
    double vh = v[k] / c2;
    double u = eps_inside_sqrt ? mh / sqrt(eps + vh) : mh / (sqrt(vh) + eps);
    theta[k] = theta[k] - lr * u - weight_decay * theta[k];
  }
  return 0;
}

/*
 * One step of the extended Adam family (Section 3.2.3, "A new family of Adam methods"; Algorithm 1).
 * All members share the first moment and differ in the preconditioner nu, built from
 *   nu_adam  = mu^2               square of the average gradient
 *   nu_micro = s^2 * sum_g2 / B   average of the per-example squares
 * through the unbiased estimators of Eq. (6):
 *   variant 0  Adam          nu = nu_adam
 *   variant 1  MicroAdam     nu = nu_micro
 *   variant 2  MicroAdamVar  nu = sigma2_hat = (nu_micro - nu_adam)     / (1 - 1/B)
 *   variant 3  MicroAdamMSQ  nu = mu2_hat    = (nu_adam  - nu_micro/B)  / (1 - 1/B)
 * (Algorithm 1 prints the factor of the last two as B/(1-B) and drops the 1/B inside MicroAdamMSQ; Eq. (6),
 * which the text says these variants implement, is followed here.)  MicroAdamMSQ clamps the bias-corrected
 * second moment at zero just before it is used (Algorithm 1; Section 3.2.3: the estimator itself stays unbiased).
 * Everything else is as in oracle_microadam_step.  Variants 2 and 3 need B >= 2.
 */
int oracle_adam_family_step(double* theta, double* m, double* v, const double* sum_g, const double* sum_g2,
                            long long n, int B, int variant, double grad_scale, double lr, double beta1,
                            double beta2, double eps, int eps_inside_sqrt, double weight_decay, int step) {
  if (!theta || !m || !v || !sum_g || !sum_g2 || n < 0 || B < 1 || step < 1) return 1;
  if (variant < 0 || variant > 3 || (variant >= 2 && B < 2)) return 1;
  double c1 = 1.0 - pow(beta1, (double)step);
  double c2 = 1.0 - pow(beta2, (double)step);
  double bessel = variant >= 2 ? 1.0 / (1.0 - 1.0 / (double)B) : 1.0;
  for (long long k = 0; k < n; ++k) {
    double mu = grad_scale * sum_g[k] / (double)B;
    double nu_adam = mu * mu;
    double nu_micro = grad_scale * grad_scale * sum_g2[k] / (double)B;
    double nu;
    switch (variant) {
      case 0: nu = nu_adam; break;
      case 1: nu = nu_micro; break;
      case 2: nu = bessel * (nu_micro - nu_adam); break;
      default: nu = bessel * (nu_adam - nu_micro / (double)B); break;
    }
    m[k] = beta1 * m[k] + (1.0 - beta1) * mu;
    v[k] = beta2 * v[k] + (1.0 - beta2) * nu;
    double mh = m[k] / c1;
    double vh = v[k] / c2;
    if (variant == 3 && vh < 0.0) vh = 0.0;
    double u = eps_inside_sqrt ? mh / sqrt(eps + vh) : mh / (sqrt(vh) + eps);
    theta[k] = theta[k] - lr * u - weight_decay * theta[k];
  }
  return 0;
}

/*
 * One MicroSignSGD step (Section 3.1: EMA o avg o sign):
 *   sbar = sum_sgn / B                       average of per-example signs
 *   m    = beta m + (1 - beta) sbar          plain EMA, no bias correction
 *   theta = theta - lr * m - wd * theta
 */
int oracle_microsignsgd_step(double* theta, double* m, const double* sum_sgn, long long n, int B,
                             double lr, double beta, double weight_decay) {
  if (!theta || !m || !sum_sgn || n < 0 || B < 1) return 1;
  for (long long k = 0; k < n; ++k) {
    double sbar = sum_sgn[k] / (double)B;
    m[k] = beta * m[k] + (1.0 - beta) * sbar;
    theta[k] = theta[k] - lr * m[k] - weight_decay * theta[k];
  }
  return 0;
}

/*
 * Sequence-level per-example statistics of a PACKED (ragged) batch: the same definition as
 * oracle_linear_stats (Section 2.3; Eq. (2)), but example b owns the token rows
 * offsets[b] .. offsets[b+1]-1 of X [rows, d_in] and dY [rows, d_out], so every gradient is contracted
 * over its own sequence's tokens, however many those are:
 *     G_b[o,i] = sum_{r = offsets[b]}^{offsets[b+1]-1} dY[r,o] * X[r,i].
 * An empty sequence has G_b = 0 (and sign(0) = 0).  offsets must be non-decreasing with offsets[0] >= 0.
 * Outputs as in oracle_linear_stats; sq_norms [B] (may be NULL) receives ||G_b||_F^2.
 */
int oracle_linear_stats_ragged(const void* X, const void* dY, int is_bf16, int B, const long long* offsets,
                               int d_in, int d_out, double small_rel, double* sum_g, double* sum_g2,
                               double* sum_sgn, double* max_abs, int32_t* n_small, double* sq_norms) {
  if (!X || !dY || !offsets || B < 0 || d_in <= 0 || d_out <= 0) return 1;
  if (B > 0 && offsets[0] < 0) return 1;
  for (int b = 0; b < B; ++b) if (offsets[b + 1] < offsets[b]) return 1;
  long long n = (long long)d_out * d_in;
  double* G = (double*)malloc(sizeof(double) * (size_t)n);
  if (!G) return 1;
  for (long long k = 0; k < n; ++k) {
    if (sum_g) sum_g[k] = 0.0;
    if (sum_g2) sum_g2[k] = 0.0;
    if (sum_sgn) sum_sgn[k] = 0.0;
    if (n_small) n_small[k] = 0;
  }
  for (int b = 0; b < B; ++b) {
    long long r0 = offsets[b], len = offsets[b + 1] - offsets[b];
    double* xb = (double*)malloc(sizeof(double) * (size_t)((len > 0 ? len : 1) * d_in));
    double* yb = (double*)malloc(sizeof(double) * (size_t)((len > 0 ? len : 1) * d_out));
    if (!xb || !yb) { free(xb); free(yb); free(G); return 1; }
    widen_rows(X, is_bf16, r0, len, d_in, xb);
    widen_rows(dY, is_bf16, r0, len, d_out, yb);
#pragma omp parallel for schedule(static)
    for (int o = 0; o < d_out; ++o) {
      double* g = G + (long long)o * d_in;
      for (int i = 0; i < d_in; ++i) g[i] = 0.0;
      for (long long t = 0; t < len; ++t) {
        double lam = yb[t * d_out + o];
        const double* h = xb + t * d_in;
        for (int i = 0; i < d_in; ++i) g[i] += lam * h[i];
      }
    }
    free(xb); free(yb);
    double mx = 0.0, nrm = 0.0;
    for (long long k = 0; k < n; ++k) {
      double a = fabs(G[k]);
      if (a > mx) mx = a;
      nrm += G[k] * G[k];
    }
    if (max_abs) max_abs[b] = mx;
    if (sq_norms) sq_norms[b] = nrm;
    for (long long k = 0; k < n; ++k) {
      double g = G[k];
      if (sum_g) sum_g[k] += g;
      if (sum_g2) sum_g2[k] += g * g;
      if (sum_sgn) sum_sgn[k] += sign3(g);
      if (n_small && fabs(g) <= small_rel * mx) n_small[k] += 1;
    }
  }
  free(G);
  return 0;
}

/*
 * Sum of norm-clipped per-example gradients (Section 2.1 lists clipping among the statistics
 * E[phi(grad f)] of Eq. (2); Section 2.3's "ghost clipping" remark names the per-example squared norms
 * N_b it needs).  The paper does not spell the clipping function out; the standard per-example L2
 * clipping is taken:
 *     c_b = min(1, C / sqrt(N_b)),      out[o,i] = sum_b c_b * G_b[o,i],      G_b = dY_b^T X_b,
 * with N_b = ||G_b||_F^2 of THIS layer when sq_norms_in is NULL, or the caller's numbers otherwise (a
 * model-wide clip passes the squared norms summed over all layers).  N_b = 0 gives c_b = 1.  The 1/B
 * of the mean is left to the caller, as everywhere else.  coef [B] (may be NULL) receives c_b.
 */
int oracle_clipped_sum(const void* X, const void* dY, int is_bf16, int B, int T, int d_in, int d_out,
                       double clip_norm, const double* sq_norms_in, double* out, double* coef) {
  if (!X || !dY || !out || B < 0 || T < 0 || d_in <= 0 || d_out <= 0 || !(clip_norm >= 0.0)) return 1;
  long long n = (long long)d_out * d_in;
  double* G = (double*)malloc(sizeof(double) * (size_t)n);
  double* xb = (double*)malloc(sizeof(double) * (size_t)((long long)(T > 0 ? T : 1) * d_in));
  double* yb = (double*)malloc(sizeof(double) * (size_t)((long long)(T > 0 ? T : 1) * d_out));
  if (!G || !xb || !yb) { free(G); free(xb); free(yb); return 1; }
  for (long long k = 0; k < n; ++k) out[k] = 0.0;
  for (int b = 0; b < B; ++b) {
    widen_rows(X, is_bf16, (long long)b * T, T, d_in, xb);
    widen_rows(dY, is_bf16, (long long)b * T, T, d_out, yb);
#pragma omp parallel for schedule(static)
    for (int o = 0; o < d_out; ++o) {
      double* g = G + (long long)o * d_in;
      for (int i = 0; i < d_in; ++i) g[i] = 0.0;
      for (int t = 0; t < T; ++t) {
        double lam = yb[(long long)t * d_out + o];
        const double* h = xb + (long long)t * d_in;
        for (int i = 0; i < d_in; ++i) g[i] += lam * h[i];
      }
    }
    double nb;
    if (sq_norms_in) {
      nb = sq_norms_in[b];
    } else {
      nb = 0.0;
      for (long long k = 0; k < n; ++k) nb += G[k] * G[k];
    }
    double norm = sqrt(nb);
    double c = (norm > clip_norm) ? clip_norm / norm : 1.0;
    if (coef) coef[b] = c;
    for (long long k = 0; k < n; ++k) out[k] += c * G[k];
  }
  free(G); free(xb); free(yb);
  return 0;
}

/* Number of OpenMP threads the loops above will use (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int oracle_num_threads(void) { return omp_get_max_threads(); }
#else
int oracle_num_threads(void) { return 1; }
#endif

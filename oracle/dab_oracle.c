/*
 * CPU checker for the DAB-Net inference hot path (arXiv 1804.02941).
 * TEST INFRASTRUCTURE ONLY: see dab_oracle.h.  Plain C, fp64, no blocking, no bit tricks.
 * Build with -ffp-contract=off so that every product, quotient and sum is rounded on its own.
 */
#include "dab_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int g_threads = 1;

void oracle_set_threads(int threads) { g_threads = threads < 1 ? 1 : threads; }
int oracle_get_threads(void) { return g_threads; }

static int cmp_double(const void* a, const void* b) {
  double x = *(const double*)a, y = *(const double*)b;
  return (x > y) - (x < y);
}

/*
 * Section 4.1: the best code for a given K takes the K smallest or the K largest values, so the
 * optimum over all masks is a threshold split of the sorted row.  Algorithm 1: sort, running prefix
 * sum P, total T, objective D_s = P_s^2/s + (T-P_s)^2/(n-s), keep the maximum with ">=".
 *
 * Readings where the text leaves a choice (each is stated in the design notes):
 *  - s runs over 1..n-1 (e != 0, e != 1 in Section 4.1; s = n would divide by zero);
 *  - the descending pass of Algorithm 1 evaluates the same set of objective values
 *    (D_desc(j) = D_asc(n-j)), so one ascending pass finds the split, and which side is
 *    called e follows "alpha captures the greater of the two values in magnitude";
 *    equal magnitudes: the high side is e;
 *  - a split is only taken between two distinct values (equal values get the same code);
 *  - a constant row is the trivial case alpha = beta of the appendix: K = 0, empty mask.
 */
void oracle_binarize_row(const float* w, int32_t n, uint8_t* e, int32_t* K, float* alpha, float* beta,
                         uint32_t* flags, int32_t* s_star, double* best_D, double* gap) {
  uint32_t fl = 0;
  int32_t i, s, sbest = 0;
  double T, P, Pbest = 0.0, best = -INFINITY, second = -INFINITY;
  double* v;

  memset(e, 0, (size_t)n);
  *K = 0;
  if (s_star) *s_star = 0;
  if (best_D) *best_D = 0.0;
  if (gap) *gap = INFINITY;

  for (i = 0; i < n; ++i)
    if (!isfinite(w[i])) fl |= ORACLE_FLAG_NONFINITE;
  if (fl & ORACLE_FLAG_NONFINITE) {
    *alpha = *beta = NAN;
    *flags = fl;
    return;
  }

  v = (double*)malloc(sizeof(double) * (size_t)n);
  for (i = 0; i < n; ++i) v[i] = (double)w[i] + 0.0; /* -0.0 becomes +0.0 */
  qsort(v, (size_t)n, sizeof(double), cmp_double);

  if (v[0] == v[n - 1]) { /* constant row, n == 1 included */
    *alpha = *beta = (float)v[0];
    *flags = fl | ORACLE_FLAG_DEGENERATE;
    free(v);
    return;
  }

  T = 0.0;
  for (i = 0; i < n; ++i) T += v[i];

  P = 0.0;
  for (s = 1; s <= n - 1; ++s) { /* s = size of the low partition */
    double Q, D;
    P += v[s - 1];
    if (v[s - 1] == v[s]) continue; /* never split a run of equal values */
    Q = T - P;
    D = (P * P) / (double)s + (Q * Q) / (double)(n - s);
    if (D >= best) { /* ">=": among exactly equal objectives the largest s wins */
      second = best;
      best = D;
      sbest = s;
      Pbest = P;
    } else if (D > second) {
      second = D;
    }
  }

  {
    double m_lo = Pbest / (double)sbest;
    double m_hi = (T - Pbest) / (double)(n - sbest);
    double t = v[sbest]; /* smallest value of the high partition */
    int32_t k = 0;
    if (fabs(m_lo) > fabs(m_hi)) { /* e marks the side whose mean is larger in magnitude */
      for (i = 0; i < n; ++i) {
        e[i] = (uint8_t)((double)w[i] < t);
        k += e[i];
      }
      *alpha = (float)m_lo;
      *beta = (float)m_hi;
    } else {
      for (i = 0; i < n; ++i) {
        e[i] = (uint8_t)((double)w[i] >= t);
        k += e[i];
      }
      *alpha = (float)m_hi;
      *beta = (float)m_lo;
    }
    *K = k;
  }
  *flags = fl;
  if (s_star) *s_star = sbest;
  if (best_D) *best_D = best;
  if (gap) *gap = (second == -INFINITY) ? INFINITY : (best - second) / best;
  free(v);
}

void oracle_binarize(const float* values, int64_t rows, int32_t n, int64_t ld_values, uint8_t* e, int32_t* K,
                     float* alpha, float* beta, uint32_t* flags, int32_t* s_star, double* best_D, double* gap) {
  int64_t r;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 16) num_threads(g_threads)
#endif
  for (r = 0; r < rows; ++r) {
    oracle_binarize_row(values + r * ld_values, n, e + r * (int64_t)n, K + r, alpha + r, beta + r, flags + r,
                        s_star ? s_star + r : 0, best_D ? best_D + r : 0, gap ? gap + r : 0);
  }
}

void oracle_sign_row(const float* w, int32_t n, uint8_t* e, int32_t* K, float* alpha, float* beta, uint32_t* flags) {
  int32_t i, k = 0;
  double sum = 0.0;
  memset(e, 0, (size_t)n);
  *K = 0;
  *flags = 0;
  for (i = 0; i < n; ++i)
    if (!isfinite(w[i])) *flags |= ORACLE_FLAG_NONFINITE;
  if (*flags) {
    *alpha = *beta = NAN;
    return;
  }
  for (i = 0; i < n; ++i) {
    sum += fabs((double)w[i]);
    e[i] = (uint8_t)((double)w[i] >= 0.0);
    k += e[i];
  }
  *K = k;
  *alpha = (float)(sum / (double)n);
  *beta = -*alpha;
}

void oracle_sign(const float* values, int64_t rows, int32_t n, int64_t ld_values, uint8_t* e, int32_t* K, float* alpha,
                 float* beta, uint32_t* flags) {
  int64_t r;
  for (r = 0; r < rows; ++r)
    oracle_sign_row(values + r * ld_values, n, e + r * (int64_t)n, K + r, alpha + r, beta + r, flags + r);
}

void oracle_pack(const uint8_t* bits, int64_t rows, int32_t n, int64_t ld_bits, uint32_t* mask, int32_t ld_mask,
                 int32_t* K) {
  int64_t r;
  for (r = 0; r < rows; ++r) {
    uint32_t* m = mask + r * (int64_t)ld_mask;
    int32_t i, k = 0;
    for (i = 0; i < ld_mask; ++i) m[i] = 0u;
    for (i = 0; i < n; ++i) {
      if (bits[r * ld_bits + i]) {
        m[i / 32] |= (uint32_t)1 << (i % 32);
        ++k;
      }
    }
    if (K) K[r] = k;
  }
}

/* One dot product of two coded rows: count the four cases, then the rescale (fp64, one final rounding). */
static float coded_dot(const uint8_t* e, float alpha, float beta, const uint8_t* f, float gamma, float delta,
                       int32_t n, int32_t* p11_out) {
  int32_t i, p11 = 0, p10 = 0, p01 = 0, p00 = 0;
  double a = (double)alpha, b = (double)beta, g = (double)gamma, d = (double)delta, y;
  for (i = 0; i < n; ++i) {
    if (e[i] && f[i]) ++p11;
    else if (e[i] && !f[i]) ++p10;
    else if (!e[i] && f[i]) ++p01;
    else ++p00;
  }
  y = (a * g) * (double)p11;
  y = y + (a * d) * (double)p10;
  y = y + (b * g) * (double)p01;
  y = y + (b * d) * (double)p00;
  if (p11_out) *p11_out = p11;
  return (float)y;
}

void oracle_gemm(int64_t M, int64_t N, int32_t n, const uint8_t* fA, const float* gamma, const float* delta,
                 const uint8_t* eB, const float* alpha, const float* beta, float* C, int32_t* p11) {
  int64_t i;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 4) num_threads(g_threads)
#endif
  for (i = 0; i < M; ++i) {
    int64_t j;
    for (j = 0; j < N; ++j) {
      C[i * N + j] = coded_dot(eB + j * (int64_t)n, alpha[j], beta[j], fA + i * (int64_t)n, gamma[i], delta[i], n,
                               p11 ? p11 + i * N + j : 0);
    }
  }
}

static void conv_out_size(const oracle_conv_desc* d, int32_t* Ho, int32_t* Wo) {
  *Ho = (d->H + 2 * d->pad_h - d->kh) / d->stride_h + 1;
  *Wo = (d->W + 2 * d->pad_w - d->kw) / d->stride_w + 1;
}

/* One patch, element order (c, kh, kw), zero padding written as 0.0 values. */
static void extract_patch(const oracle_conv_desc* d, const float* x, int32_t img, int32_t ho, int32_t wo, float* p) {
  int32_t c, r, s, idx = 0;
  for (c = 0; c < d->C; ++c)
    for (r = 0; r < d->kh; ++r)
      for (s = 0; s < d->kw; ++s) {
        int32_t h = ho * d->stride_h - d->pad_h + r;
        int32_t w = wo * d->stride_w - d->pad_w + s;
        float v = 0.0f;
        if (h >= 0 && h < d->H && w >= 0 && w < d->W) v = x[(((int64_t)img * d->C + c) * d->H + h) * d->W + w];
        p[idx++] = v;
      }
}

void oracle_im2col(const oracle_conv_desc* d, const float* x, float* patches) {
  int32_t Ho, Wo, img, ho, wo;
  int32_t n = d->C * d->kh * d->kw;
  conv_out_size(d, &Ho, &Wo);
  for (img = 0; img < d->N; ++img)
    for (ho = 0; ho < Ho; ++ho)
      for (wo = 0; wo < Wo; ++wo)
        extract_patch(d, x, img, ho, wo, patches + (((int64_t)img * Ho + ho) * Wo + wo) * n);
}

static void conv_with_coder(int sign_coder, const oracle_conv_desc* d, const float* x, const uint8_t* w_e,
                            const float* w_alpha, const float* w_beta, float* y, uint8_t* p_e, int32_t* p_K,
                            float* p_gamma, float* p_delta, uint32_t* p_flags, int32_t* p_p11) {
  int32_t Ho, Wo;
  int32_t n = d->C * d->kh * d->kw;
  int64_t patches, pi;
  conv_out_size(d, &Ho, &Wo);
  patches = (int64_t)d->N * Ho * Wo;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 8) num_threads(g_threads)
#endif
  for (pi = 0; pi < patches; ++pi) {
    int32_t img = (int32_t)(pi / ((int64_t)Ho * Wo));
    int32_t ho = (int32_t)((pi / Wo) % Ho);
    int32_t wo = (int32_t)(pi % Wo);
    float* p = (float*)malloc(sizeof(float) * (size_t)n);
    uint8_t* f = (uint8_t*)malloc((size_t)n);
    int32_t Kf, co;
    float gamma, delta;
    uint32_t fl;
    extract_patch(d, x, img, ho, wo, p);
    if (sign_coder) oracle_sign_row(p, n, f, &Kf, &gamma, &delta, &fl);
    else oracle_binarize_row(p, n, f, &Kf, &gamma, &delta, &fl, 0, 0, 0);
    if (p_e) memcpy(p_e + pi * (int64_t)n, f, (size_t)n);
    if (p_K) p_K[pi] = Kf;
    if (p_gamma) p_gamma[pi] = gamma;
    if (p_delta) p_delta[pi] = delta;
    if (p_flags) p_flags[pi] = fl;
    for (co = 0; co < d->Cout; ++co) {
      int32_t p11;
      float out = coded_dot(w_e + (int64_t)co * n, w_alpha[co], w_beta[co], f, gamma, delta, n, &p11);
      y[(((int64_t)img * d->Cout + co) * Ho + ho) * Wo + wo] = out;
      if (p_p11) p_p11[pi * d->Cout + co] = p11;
    }
    free(p);
    free(f);
  }
}

void oracle_conv(const oracle_conv_desc* d, const float* x, const uint8_t* w_e, const float* w_alpha,
                 const float* w_beta, float* y, uint8_t* p_e, int32_t* p_K, float* p_gamma, float* p_delta,
                 uint32_t* p_flags, int32_t* p_p11) {
  conv_with_coder(0, d, x, w_e, w_alpha, w_beta, y, p_e, p_K, p_gamma, p_delta, p_flags, p_p11);
}

void oracle_conv_sign(const oracle_conv_desc* d, const float* x, const uint8_t* w_e, const float* w_alpha,
                      const float* w_beta, float* y, uint8_t* p_e, int32_t* p_K, float* p_gamma, float* p_delta,
                      uint32_t* p_flags, int32_t* p_p11) {
  conv_with_coder(1, d, x, w_e, w_alpha, w_beta, y, p_e, p_K, p_gamma, p_delta, p_flags, p_p11);
}

/* Section 4.3.2, weights-only binarization: the plain convolution of the fp32 input with the two-level
 * filters W~ = alpha*e + beta*(1-e).  Every product and the running sum are fp64, in element order
 * (c, kh, kw); one rounding to fp32 at the end. */
void oracle_conv_wbin(const oracle_conv_desc* d, const float* x, const uint8_t* w_e, const float* w_alpha,
                      const float* w_beta, float* y, double* abs_terms) {
  int32_t Ho, Wo;
  int32_t n = d->C * d->kh * d->kw;
  int64_t patches, pi;
  conv_out_size(d, &Ho, &Wo);
  patches = (int64_t)d->N * Ho * Wo;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 8) num_threads(g_threads)
#endif
  for (pi = 0; pi < patches; ++pi) {
    int32_t img = (int32_t)(pi / ((int64_t)Ho * Wo));
    int32_t ho = (int32_t)((pi / Wo) % Ho);
    int32_t wo = (int32_t)(pi % Wo);
    float* p = (float*)malloc(sizeof(float) * (size_t)n);
    int32_t co, i;
    extract_patch(d, x, img, ho, wo, p);
    for (co = 0; co < d->Cout; ++co) {
      const uint8_t* e = w_e + (int64_t)co * n;
      double a = (double)w_alpha[co], b = (double)w_beta[co], acc = 0.0, mag = 0.0;
      int64_t o = (((int64_t)img * d->Cout + co) * Ho + ho) * Wo + wo;
      for (i = 0; i < n; ++i) {
        double t = (double)p[i] * (e[i] ? a : b);
        acc = acc + t;
        mag = mag + fabs(t);
      }
      y[o] = (float)acc;
      if (abs_terms) abs_terms[o] = mag;
    }
    free(p);
  }
}

/* Algorithm 2, steps 4-13 for the filters of one layer: MeanCenter (the mean of the filter's n weights is
 * subtracted), Clamp to [-1, 1], then Algorithm 1 and the dense two-level filter of Corollary 1. */
void oracle_train_forward(const float* W, int64_t rows, int32_t n, float* Wc, uint8_t* e, int32_t* K, float* alpha,
                          float* beta, uint32_t* flags, float* Wt) {
  int64_t r;
  for (r = 0; r < rows; ++r) {
    const float* w = W + r * (int64_t)n;
    float* c = Wc + r * (int64_t)n;
    double sum = 0.0, mean;
    int32_t i;
    for (i = 0; i < n; ++i) sum = sum + (double)w[i];
    mean = sum / (double)n;
    for (i = 0; i < n; ++i) {
      float v = (float)((double)w[i] - mean);
      if (v > 1.0f) v = 1.0f;
      if (v < -1.0f) v = -1.0f;
      c[i] = v;
    }
    oracle_binarize_row(c, n, e + r * (int64_t)n, K + r, alpha + r, beta + r, flags + r, 0, 0, 0);
    if (Wt)
      for (i = 0; i < n; ++i) Wt[r * (int64_t)n + i] = e[r * (int64_t)n + i] ? alpha[r] : beta[r];
  }
}

/* Theorem 4, element by element, for rows W (the mean-centred, clamped weights that were coded) with masks e:
 *   T_k = W o e (the selected weights, zeros elsewhere), sgn(T_k) read as the membership indicator e,
 *   sgn(W - T_k) as 1 - e, STE(V)_i = V_i where |W_i| <= 1 and 0 elsewhere;
 *   G1_i = e_i / K + (||T_k||_1 / K) * STE(T_k)_i
 *   G2_i = (1 - e_i) / (n - K) + (||W - T_k||_1 / (n - K)) * STE(W - T_k)_i
 *   G = G1 + G2 (fp64).  Rows with K = 0 (constant rows) get G = 0.
 * grad_W (nullable) = grad_Wt o G rounded to fp32: the gradient handed to the weight update. */
void oracle_theorem4(const float* W, const uint8_t* e, const int32_t* K, int64_t rows, int32_t n, double* G,
                     const float* grad_Wt, float* grad_W) {
  int64_t r;
  for (r = 0; r < rows; ++r) {
    const float* w = W + r * (int64_t)n;
    const uint8_t* m = e + r * (int64_t)n;
    double l1_sel = 0.0, l1_rest = 0.0;
    int32_t i, k = K[r];
    for (i = 0; i < n; ++i) {
      if (m[i]) l1_sel = l1_sel + fabs((double)w[i]);
      else l1_rest = l1_rest + fabs((double)w[i]);
    }
    for (i = 0; i < n; ++i) {
      double g = 0.0;
      if (k > 0 && k < n) {
        double ste = (fabs((double)w[i]) <= 1.0) ? (double)w[i] : 0.0;
        if (m[i]) g = 1.0 / (double)k + (l1_sel / (double)k) * ste;
        else g = 1.0 / (double)(n - k) + (l1_rest / (double)(n - k)) * ste;
      }
      if (G) G[r * (int64_t)n + i] = g;
      if (grad_W) grad_W[r * (int64_t)n + i] = (float)((double)grad_Wt[r * (int64_t)n + i] * g);
    }
  }
}

/* ------------------------------------------------------------------------------------------------------------
 * Full-precision layers around the binarized ones (Section 5.1), plain definitions.
 * ------------------------------------------------------------------------------------------------------------ */
void oracle_conv_dense(const oracle_conv_desc* d, const float* x, const float* w, const float* bias, float* y) {
  int32_t Ho, Wo;
  int64_t outputs, oi;
  int32_t n = d->C * d->kh * d->kw;
  conv_out_size(d, &Ho, &Wo);
  outputs = (int64_t)d->N * d->Cout * Ho * Wo;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(g_threads)
#endif
  for (oi = 0; oi < outputs; ++oi) {
    int32_t wo = (int32_t)(oi % Wo);
    int32_t ho = (int32_t)((oi / Wo) % Ho);
    int32_t co = (int32_t)((oi / ((int64_t)Wo * Ho)) % d->Cout);
    int32_t img = (int32_t)(oi / ((int64_t)Wo * Ho * d->Cout));
    double acc = 0.0;
    int32_t c, r, s;
    for (c = 0; c < d->C; ++c)
      for (r = 0; r < d->kh; ++r)
        for (s = 0; s < d->kw; ++s) {
          int32_t h = ho * d->stride_h - d->pad_h + r, wq = wo * d->stride_w - d->pad_w + s;
          double xv = 0.0, prod;
          if (h >= 0 && h < d->H && wq >= 0 && wq < d->W) xv = (double)x[(((int64_t)img * d->C + c) * d->H + h) * d->W + wq];
          prod = xv * (double)w[(int64_t)co * n + ((int64_t)c * d->kh + r) * d->kw + s];
          acc = acc + prod;
        }
    if (bias) acc = acc + (double)bias[co];
    y[oi] = (float)acc;
  }
}

void oracle_affine(const float* x, int64_t N, int32_t C, int64_t HW, const float* scale, const float* shift, float* y) {
  int64_t total = N * C * HW, i;
  for (i = 0; i < total; ++i) {
    int32_t c = (int32_t)((i / HW) % C);
    double t = (double)scale[c] * (double)x[i];
    y[i] = (float)(t + (double)shift[c]);
  }
}

void oracle_relu(const float* x, int64_t count, float* y) {
  int64_t i;
  for (i = 0; i < count; ++i) y[i] = x[i] > 0.0f ? x[i] : 0.0f;
}

void oracle_maxpool(const oracle_conv_desc* d, const float* x, float* y) {
  int32_t Ho, Wo;
  int64_t outputs, oi;
  conv_out_size(d, &Ho, &Wo);
  outputs = (int64_t)d->N * d->C * Ho * Wo;
  for (oi = 0; oi < outputs; ++oi) {
    int32_t wo = (int32_t)(oi % Wo);
    int32_t ho = (int32_t)((oi / Wo) % Ho);
    int64_t plane = oi / ((int64_t)Wo * Ho);
    int32_t r, s, seen = 0;
    float best = 0.0f;
    for (r = 0; r < d->kh; ++r)
      for (s = 0; s < d->kw; ++s) {
        int32_t h = ho * d->stride_h - d->pad_h + r, wq = wo * d->stride_w - d->pad_w + s;
        if (h >= 0 && h < d->H && wq >= 0 && wq < d->W) {
          float v = x[(plane * d->H + h) * d->W + wq];
          if (!seen || v > best) best = v;
          seen = 1;
        }
      }
    y[oi] = best;
  }
}

void oracle_add(const float* a, const float* b, int64_t count, float* y) {
  int64_t i;
  for (i = 0; i < count; ++i) y[i] = a[i] + b[i];
}

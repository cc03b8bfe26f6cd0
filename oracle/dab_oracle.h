/*
 * CPU checker for the DAB-Net inference hot path (arXiv 1804.02941).
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, fp64 restatement of what the
 * paper defines: it exists so that the CUDA library can be compared against
 * something written independently.  It shares no code, table, constant or helper
 * with the CUDA library and must never be called from a product code path; only
 * the test-suite, the smoke check and the CPU-baseline leg of the benchmark use it.
 *
 * Every function below is pinned by CPU tests against something other than
 * itself (exhaustive search over all masks, direct sums of squared error, closed
 * forms, a library im2col, a textbook XNOR-popcount).  One exception, marked "PARITY UNPINNED" at its
 * declaration: the straight-through terms of oracle_theorem4.
 */
#ifndef DAB_ORACLE_H
#define DAB_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ORACLE_FLAG_DEGENERATE 1u /* all values of the row are equal (includes n == 1) */
#define ORACLE_FLAG_NONFINITE 2u  /* a NaN or an infinity was seen; the other outputs are unspecified */

/* Number of worker threads used by the batched functions (rows are independent). */
void oracle_set_threads(int threads);
int oracle_get_threads(void);

/*
 * Section 4.1 + Algorithm 1: best two-level code  W~ = alpha*e + beta*(1-e)  of one row.
 *   w[n]        fp32 values
 *   e[n]        out, 0/1 bytes (unpacked mask)
 *   K           out, number of ones in e
 *   alpha,beta  out, partition means rounded once to fp32
 *   flags       out, ORACLE_FLAG_*
 *   s_star      out (nullable), size of the low partition at the chosen split
 *   best_D      out (nullable), objective value at the chosen split
 *   gap         out (nullable), (best - second best objective) / best over the evaluated splits,
 *               +inf when fewer than two splits were evaluated
 */
void oracle_binarize_row(const float* w, int32_t n, uint8_t* e, int32_t* K, float* alpha, float* beta,
                         uint32_t* flags, int32_t* s_star, double* best_D, double* gap);

/* The same for `rows` rows, row r starting at values + r*ld_values; e is rows x n bytes, dense.
 * s_star, best_D, gap nullable. */
void oracle_binarize(const float* values, int64_t rows, int32_t n, int64_t ld_values, uint8_t* e, int32_t* K,
                     float* alpha, float* beta, uint32_t* flags, int32_t* s_star, double* best_D, double* gap);

/*
 * Sign coding with one scale (the XNOR-Net code the paper's fully binarized layers use for their inputs,
 * Appendix "Experimental details"; the special case alpha = -beta of Section 4.1):
 *   e_i = [w_i >= 0], alpha = mean |w_i|, beta = -alpha, K = number of ones.  -0.0 counts as +0.0.
 * flags: ORACLE_FLAG_NONFINITE as above (then alpha = beta = NaN, empty mask); no row is degenerate here.
 */
void oracle_sign_row(const float* w, int32_t n, uint8_t* e, int32_t* K, float* alpha, float* beta, uint32_t* flags);
void oracle_sign(const float* values, int64_t rows, int32_t n, int64_t ld_values, uint8_t* e, int32_t* K, float* alpha,
                 float* beta, uint32_t* flags);

/* Bit packing: bit (i mod 32) of word (i div 32) of a row is e_i; words up to ld_mask and bits beyond n are 0.
 * K (nullable) receives the number of ones per row. */
void oracle_pack(const uint8_t* bits, int64_t rows, int32_t n, int64_t ld_bits, uint32_t* mask, int32_t ld_mask,
                 int32_t* K);

/*
 * Dot products of two-level coded rows.  A side: masks fA (M x n bytes), scalars gamma/delta.
 * B side: masks eB (N x n bytes), scalars alpha/beta.  For every (i, j) the four cases
 * (e,f) = (1,1), (1,0), (0,1), (0,0) are counted element by element and
 *   C[i,j] = alpha*gamma*p11 + alpha*delta*p10 + beta*gamma*p01 + beta*delta*p00
 * is evaluated in fp64 from the fp32 scalars and rounded once to fp32.
 * p11 (nullable, M x N) receives the (1,1) counts.
 */
void oracle_gemm(int64_t M, int64_t N, int32_t n, const uint8_t* fA, const float* gamma, const float* delta,
                 const uint8_t* eB, const float* alpha, const float* beta, float* C, int32_t* p11);

typedef struct {
  int32_t N, C, H, W, Cout, kh, kw, stride_h, stride_w, pad_h, pad_w;
} oracle_conv_desc;

/*
 * Section 4.3.2 forward pass  I (*) W~  with every input patch coded by oracle_binarize_row.
 *   x        N x C x H x W fp32
 *   w_e      Cout x (C*kh*kw) 0/1 bytes, element order (c, kh, kw); w_alpha, w_beta per filter
 *   y        N x Cout x Ho x Wo fp32
 * Optional per-patch outputs, patch index = (img*Ho + ho)*Wo + wo (all nullable):
 *   p_e (patches x n bytes), p_K, p_gamma, p_delta, p_flags, p_p11 (patches x Cout)
 * Zero padding is part of the patch: padded positions are 0.0 values like any other.
 */
void oracle_conv(const oracle_conv_desc* d, const float* x, const uint8_t* w_e, const float* w_alpha,
                 const float* w_beta, float* y, uint8_t* p_e, int32_t* p_K, float* p_gamma, float* p_delta,
                 uint32_t* p_flags, int32_t* p_p11);

/* The same forward pass with every input patch coded by oracle_sign_row instead (paper-faithful FBin inputs). */
void oracle_conv_sign(const oracle_conv_desc* d, const float* x, const uint8_t* w_e, const float* w_alpha,
                      const float* w_beta, float* y, uint8_t* p_e, int32_t* p_K, float* p_gamma, float* p_delta,
                      uint32_t* p_flags, int32_t* p_p11);

/*
 * Section 4.3.2 forward pass with weights-only binarization (the paper's WBin networks): the fp32 input is
 * convolved with the two-level filters W~ = alpha*e + beta*(1-e); nothing is done to the activations.
 *   y[img][co][ho][wo] = sum over (c, kh, kw) of x_patch[i] * (e_co[i] ? alpha_co : beta_co)
 * Products and the running sum are fp64, elements taken in (c, kh, kw) order, one rounding to fp32.
 * abs_terms (nullable, same shape as y, fp64) receives the sum of |product|: the scale rounding errors of any
 * other summation order are measured against.
 */
void oracle_conv_wbin(const oracle_conv_desc* d, const float* x, const uint8_t* w_e, const float* w_alpha,
                      const float* w_beta, float* y, double* abs_terms);

/*
 * Algorithm 2, steps 4-13 (binarizing the weight filters of one layer during training):
 *   Wc = Clamp(MeanCenter(W), -1, 1): the mean of each filter's n weights (fp64 sum in element order, divided by
 *   n) is subtracted in fp64, the difference rounded to fp32 and clamped;  (e, K, alpha, beta) = Algorithm 1 on Wc;
 *   Wt (nullable) = alpha e + beta (1 - e), the dense filter of Corollary 1.  All arrays rows x n, dense.
 */
void oracle_train_forward(const float* W, int64_t rows, int32_t n, float* Wc, uint8_t* e, int32_t* K, float* alpha,
                          float* beta, uint32_t* flags, float* Wt);

/*
 * Theorem 4 (backward pass), element by element; W is the mean-centred, clamped weight matrix that was coded.
 *   G (nullable, fp64, rows x n) = G1 + G2 as printed, with sgn(T_k) read as the membership indicator e;
 *   grad_W (nullable) = grad_Wt o G rounded to fp32.  See the comment in the source for every term.
 * PARITY UNPINNED for the two STE terms: the paper prints them without a definition they could be checked
 * against (they are not the derivative of anything the paper defines); the other two terms are pinned as the
 * derivatives of alpha and beta with e held fixed.
 */
void oracle_theorem4(const float* W, const uint8_t* e, const int32_t* K, int64_t rows, int32_t n, double* G,
                     const float* grad_Wt, float* grad_W);

/* Patch extraction alone (explicit loops), rows = N*Ho*Wo, row length C*kh*kw. */
void oracle_im2col(const oracle_conv_desc* d, const float* x, float* patches);

/*
 * The layers around the binarized ones when whole networks are chained (Section 5.1: the first layer, and the last
 * one in Sketch-A-Net, stay full precision; Appendix "Experimental details" for the glue).  The paper gives no
 * arithmetic for them; each is written here as its plain definition, fp64 inside, one rounding to fp32.
 *
 * oracle_conv_dense  y = x (*) W (+ bias): for every output the products are summed in fp64 in element order
 *                    (c, kh, kw), each product and sum rounded on its own, zero padding; W is [Cout][C*kh*kw].
 * oracle_affine      y = scale[c] * x + shift[c] per channel (a folded normalisation layer); x is N x C x HW.
 * oracle_relu        y = x > 0 ? x : 0  (-0.0 and NaN give +0.0).
 * oracle_maxpool     maximum over the kh x kw window (positions outside the image are skipped); d->C channels,
 *                    d->Cout ignored; output size as for a convolution of the same geometry.
 * oracle_add         y = a + b in fp32 (the shortcut of a residual block).
 */
void oracle_conv_dense(const oracle_conv_desc* d, const float* x, const float* w, const float* bias, float* y);
void oracle_affine(const float* x, int64_t N, int32_t C, int64_t HW, const float* scale, const float* shift, float* y);
void oracle_relu(const float* x, int64_t count, float* y);
void oracle_maxpool(const oracle_conv_desc* d, const float* x, float* y);
void oracle_add(const float* a, const float* b, int64_t count, float* y);

#ifdef __cplusplus
}
#endif
#endif

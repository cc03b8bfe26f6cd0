/*
 * libdab — distribution-aware binarization (DAB-Net, arXiv 1804.02941) inference hot path for
 * NVIDIA B200 (sm_100a).  C ABI: plain pointers and sizes, no C++ or framework types.
 *
 * Vocabulary (paper, Section 4.1): a row W in R^n (a flattened weight filter, n = c*w*h, or an
 * activation patch in the same element order) is coded as  W~ = alpha*e + beta*(1-e),
 * e in {0,1}^n, K = e^T e.  The weight side of a contraction carries (e, K_e, alpha, beta), the
 * activation side (f, K_f, gamma, delta).
 *
 * Conventions for every entry point
 *   - Pointers named d_* are DEVICE pointers owned by the caller; h_* are HOST pointers.  The
 *     library allocates and frees no device memory.  What it keeps between calls is listed under
 *     "State" below; none of it carries data from one call's inputs to another call's outputs.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls enqueue
 *     work on that stream and return without synchronising, except where stated.
 *   - Errors are return codes.  Arguments are validated on the host before anything is
 *     launched; nothing aborts, traps or throws.  There is no CPU fallback.
 *   - Packed masks: 32-bit words, element i of a row is bit (i mod 32) of word (i div 32).  A row
 *     occupies ld words, ld >= ceil(n/32) and ld % 4 == 0, base pointer 16-byte aligned.  Bits
 *     beyond n and words beyond ceil(n/32) are written as 0 by the producers and must be 0 for
 *     the consumers.
 *   - Row length limit: 1 <= n <= DAB_MAX_N.
 *
 * State kept by the library (process-wide unless stated; every item is safe to use from several threads)
 *   - the patch-coder and contraction choices (dab_set_patch_coder, dab_set_contraction): atomic integers
 *     read once at the start of each call;
 *   - per device: the SM count and, per kernel, the largest dynamic shared-memory size it was opted in to
 *     (caches of driver queries, behind a mutex);
 *   - per device: two copy streams and a few events of dab_binary_conv_host, created on its first call;
 *     calls of that entry point on one device are serialised by a lock;
 *   - per device: the address of dab_binary_conv_static's scratch array, and the array itself, which keeps
 *     the last call's patch codes (see that entry point);
 *   - per device: two counters of barrier waits that ran out (dab_contraction_wait_failures).
 *   Cached device addresses do not survive cudaDeviceReset: do not reset a device while the library is loaded.
 *   Calls on different streams may run concurrently; kernels of one call hand work to each other only through
 *   that call's own output arrays.
 */
#ifndef DAB_H
#define DAB_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DAB_MAX_N 16384

typedef enum {
  DAB_OK = 0,
  DAB_ERR_INVALID_ARG = 1, /* null pointer, negative size, bad stride or alignment */
  DAB_ERR_UNSUPPORTED = 2, /* a size beyond a documented limit */
  DAB_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small */
  DAB_ERR_CUDA = 4         /* a CUDA runtime call or a kernel launch failed */
} dab_status;

#define DAB_ROW_DEGENERATE 1u /* all values of the row are equal (n == 1 included): K = 0, empty mask, alpha = beta */
#define DAB_ROW_NONFINITE 2u  /* a NaN or an infinity was seen: K = 0, empty mask, alpha = beta = NaN */

const char* dab_status_string(dab_status s);
int32_t dab_words_per_row(int32_t n); /* ceil(n/32) */
int32_t dab_default_ld(int32_t n);    /* dab_words_per_row rounded up to a multiple of 4 words (16 bytes) */

/*
 * dab_binarize — optimal two-level code of every row (Section 4.1 "Derivation"; Algorithm 1
 * "Finding an optimal K value"; Section 4.3.1 on treating all filters as one 2-D array).
 *
 * For each row: sort, prefix sums P_s, total T, objective D_s = P_s^2/s + (T-P_s)^2/(n-s) over the
 * splits s = 1..n-1 that fall between two distinct values, maximum with ">=" (the largest s wins
 * exact ties).  The low partition has mean m_lo = P_s/s, the high one m_hi = (T-P_s)/(n-s).  e marks
 * the partition whose mean is larger in magnitude (the high one when equal); alpha is that mean,
 * beta the other.  All of it in fp64; alpha and beta are rounded once to fp32.  -0.0 counts as +0.0.
 *
 *   d_values    rows x n fp32, row r at d_values + r*ld_values (ld_values >= n)
 *   d_K         out, rows int32
 *   d_alpha     out, rows fp32;  d_beta likewise
 *   d_mask      out, rows x ld_mask words (see "Packed masks")
 *   d_row_flags out, rows uint32 of DAB_ROW_* bits; may be NULL
 * rows == 0 is a no-op returning DAB_OK.
 */
dab_status dab_binarize(const float* d_values, int64_t rows, int32_t n, int64_t ld_values, int32_t* d_K,
                        float* d_alpha, float* d_beta, uint32_t* d_mask, int32_t ld_mask, uint32_t* d_row_flags,
                        void* stream);

/*
 * dab_pack — 0/1 bytes to packed words (the mask e of Section 4.1 in the bit layout above; any
 * non-zero byte counts as 1).
 *   d_bits  rows x n bytes, row r at d_bits + r*ld_bits (ld_bits >= n)
 *   d_mask  out, rows x ld_mask words
 *   d_K     out, rows int32 = number of ones per row; may be NULL
 */
dab_status dab_pack(const uint8_t* d_bits, int64_t rows, int32_t n, int64_t ld_bits, uint32_t* d_mask,
                    int32_t ld_mask, int32_t* d_K, void* stream);

/*
 * dab_binary_gemm — all dot products between M activation-side rows and N weight-side rows of
 * two-level codes.  With W~ = alpha e + beta(1-e) (Section 4.1) and X~ = gamma f + delta(1-f), the
 * forward product of Section 4.3.2 expands over the four 0/1 indicator pairs:
 *   C[i,j] = alpha_j gamma_i p11 + alpha_j delta_i p10 + beta_j gamma_i p01 + beta_j delta_i p00,
 *   p11 = popc(e_j & f_i), p10 = K_e - p11, p01 = K_f - p11, p00 = n - K_e - K_f + p11
 * evaluated in fp64 from the fp32 scalars in exactly that order of terms, rounded once to fp32.
 *
 *   d_A, lda, d_KA, d_gamma, d_delta   activation side: M packed rows, their K_f, gamma, delta
 *   d_B, ldb, d_KB, d_alpha, d_beta    weight side: N packed rows, their K_e, alpha, beta
 *   d_C, ldc                           out, row-major M x N fp32, row stride ldc >= N
 *   d_p11, ldp                         out, raw AND-popcounts (int32, row stride ldp >= N); may be NULL
 */
dab_status dab_binary_gemm(int64_t M, int64_t N, int32_t n, const uint32_t* d_A, int32_t lda, const int32_t* d_KA,
                           const float* d_gamma, const float* d_delta, const uint32_t* d_B, int32_t ldb,
                           const int32_t* d_KB, const float* d_alpha, const float* d_beta, float* d_C, int64_t ldc,
                           int32_t* d_p11, int64_t ldp, void* stream);

typedef struct {
  int32_t N, C, H, W;     /* input, NCHW fp32 */
  int32_t Cout, kh, kw;   /* filters, each flattened in (c, kh, kw) order: n = C*kh*kw */
  int32_t stride_h, stride_w, pad_h, pad_w;
} dab_conv_desc;

/* Output extent of a convolution; returns DAB_ERR_INVALID_ARG for an impossible geometry. */
dab_status dab_conv_output_size(const dab_conv_desc* desc, int32_t* Ho, int32_t* Wo);

/* Bytes of scratch dab_binary_conv needs for this geometry (0 if the descriptor is invalid). */
size_t dab_binary_conv_workspace(const dab_conv_desc* desc);

/*
 * dab_binary_conv — the binary forward pass I (*) W~ of Section 4.3.2 with every input patch coded
 * like a filter: each patch (the C*kh*kw values under one output position, element order (c, kh, kw),
 * zero padding present as 0.0 values) is binarized as in dab_binarize, then contracted with every
 * pre-binarized filter as in dab_binary_gemm.  No bias (the paper's binarized layers have none).
 *
 *   d_x                          N x C x H x W fp32
 *   d_wmask, ldw, d_wK, d_walpha, d_wbeta   the filters as written by dab_binarize on [Cout x C*kh*kw]
 *   d_y                          out, N x Cout x Ho x Wo fp32
 *   d_workspace, workspace_bytes scratch of at least dab_binary_conv_workspace(desc) bytes, 256-byte aligned
 * Optional outputs (each may be NULL), patch index p = (img*Ho + ho)*Wo + wo:
 *   d_pK, d_pgamma, d_pdelta     per-patch K_f, gamma, delta
 *   d_pmask, ldp                 per-patch packed masks, ldp words apart
 *   d_pflags                     per-patch DAB_ROW_* bits
 *   d_p11                        raw AND-popcounts, patches x Cout int32
 */
dab_status dab_binary_conv(const dab_conv_desc* desc, const float* d_x, const uint32_t* d_wmask, int32_t ldw,
                           const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* d_y,
                           void* d_workspace, size_t workspace_bytes, int32_t* d_pK, float* d_pgamma,
                           float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, int32_t* d_p11,
                           void* stream);

/*
 * The two stages of dab_binary_conv as calls of their own (dab_binary_conv runs exactly these two, in this
 * order, on the same stream).  A caller that wants the patch codes of an activation tensor once and several
 * contractions against them, or that times the stages separately, uses these.
 *
 * dab_binarize_patches — Section 4.1 / Algorithm 1 applied to every patch of d_x (patch definition, element
 * order and zero padding as in dab_binary_conv); outputs as the optional outputs of dab_binary_conv, here
 * required except d_pflags.
 *
 * dab_binary_conv_contract — Section 4.3.2: the coded patches against the coded filters, result in NCHW.
 * d_p11 (patches x Cout int32) may be NULL.
 */
dab_status dab_binarize_patches(const dab_conv_desc* desc, const float* d_x, int32_t* d_pK, float* d_pgamma,
                                float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, void* stream);
dab_status dab_binary_conv_contract(const dab_conv_desc* desc, const uint32_t* d_pmask, int32_t ldp,
                                    const int32_t* d_pK, const float* d_pgamma, const float* d_pdelta,
                                    const uint32_t* d_wmask, int32_t ldw, const int32_t* d_wK, const float* d_walpha,
                                    const float* d_wbeta, float* d_y, int32_t* d_p11, void* stream);

/*
 * Sign coding — the input coding of the paper's fully binarized ("FBin") layers, which are "structured the same
 * as the XNOR-Net" (Appendix, "Experimental details"): mask bit = [x >= 0], gamma = mean |x| over the row,
 * delta = -gamma.  It is the special case alpha = -beta of Section 4.1 (no search, no sort).  Outputs have the
 * layout of dab_binarize / dab_binarize_patches, so the contraction calls take them unchanged.  -0.0 counts as
 * +0.0; rows with a NaN or an infinity get DAB_ROW_NONFINITE, K = 0, an empty mask and NaN scales.
 *
 * dab_sign_binarize        rows of a matrix (arguments as dab_binarize)
 * dab_sign_patches         patches of an NCHW tensor (arguments as dab_binarize_patches)
 * dab_binary_conv_sign     dab_sign_patches + dab_binary_conv_contract (arguments as dab_binary_conv)
 */
dab_status dab_sign_binarize(const float* d_values, int64_t rows, int32_t n, int64_t ld_values, int32_t* d_K,
                             float* d_alpha, float* d_beta, uint32_t* d_mask, int32_t ld_mask, uint32_t* d_row_flags,
                             void* stream);
dab_status dab_sign_patches(const dab_conv_desc* desc, const float* d_x, int32_t* d_pK, float* d_pgamma,
                            float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, void* stream);
dab_status dab_binary_conv_sign(const dab_conv_desc* desc, const float* d_x, const uint32_t* d_wmask, int32_t ldw,
                                const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* d_y,
                                void* d_workspace, size_t workspace_bytes, int32_t* d_pK, float* d_pgamma,
                                float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, int32_t* d_p11,
                                void* stream);

/*
 * dab_wbin_conv — Section 4.3.2 / Corollary 1 as the paper's weights-only ("WBin") networks run it: the
 * full-precision input convolved with the two-level filters W~ = alpha e + beta (1 - e),
 *   y[img][co][ho][wo] = alpha_co * (sum of the patch values under e_co) + beta_co * (sum of the others),
 * with nothing done to the activations.  Patch definition, element order (c, kh, kw), zero padding and output
 * layout as in dab_binary_conv; the filters come from dab_binarize on the [Cout x C*kh*kw] weight matrix
 * (their K is not needed).
 *   d_workspace, workspace_bytes   scratch of at least dab_wbin_conv_workspace(desc) bytes (one word per input
 *                                  pixel: the largest magnitude over its channels), 256-byte aligned
 *
 * Arithmetic: each patch is taken as 32-bit fixed point relative to its own largest magnitude and the sums
 * under e are formed exactly in integers on the tensor cores, so the result differs from exact arithmetic by
 * at most 2^-32 * n * max|x_patch| * max(|alpha|, |beta|) plus the final rounding to fp32 (patches whose largest
 * magnitude is subnormal are resolved to 2^-158 instead).  A patch that contains a NaN or an infinity gives NaN
 * in all its outputs.  C*H*W must be below 2^31.
 * DAB_ERR_UNSUPPORTED if no tile of the layer fits shared memory (kernels wider than about 200 columns).
 */
size_t dab_wbin_conv_workspace(const dab_conv_desc* desc);
dab_status dab_wbin_conv(const dab_conv_desc* desc, const float* d_x, const uint32_t* d_wmask, int32_t ldw,
                         const float* d_walpha, const float* d_wbeta, float* d_y, void* d_workspace,
                         size_t workspace_bytes, void* stream);

/*
 * dab_binarize_train — Algorithm 2, steps 4-13: how the filters of a layer are binarized at every training
 * step.  For each row (filter) of d_W:
 *   Wc = Clamp(MeanCenter(W), -1, 1)   the mean of the row's n weights (fp64) is subtracted, the result rounded
 *                                      to fp32 and clamped; Wc is what Algorithm 2 keeps as W_real and what is coded
 *   (e, K, alpha, beta) = Algorithm 1 on Wc, exactly as dab_binarize
 *   Wt = alpha e + beta (1 - e)        the dense filter of Corollary 1 (d_Wt may be NULL)
 * d_W, d_Wc, d_Wt: rows x n fp32 with row strides ld_* (floats); d_Wc may not alias d_W unless ld_Wc == ld_W
 * (then the update is in place).  The other arguments are those of dab_binarize.
 *
 * dab_binarize_backward — Theorem 4: grad_W = grad_Wt o G, the gradient handed to the weight update, with
 *   G_i = e_i / K + (||T_k||_1 / K) STE(T_k)_i + (1 - e_i) / (n - K) + (||W - T_k||_1 / (n - K)) STE(W - T_k)_i,
 * T_k = Wc o e, STE(V)_i = V_i where |Wc_i| <= 1 and 0 elsewhere, sgn(T_k) of the printed formula read as the
 * membership indicator e.  d_Wc, d_mask, d_K are the outputs of dab_binarize_train; rows with K = 0 (constant
 * rows) get a zero gradient.  fp64 internally, one rounding to fp32.
 */
dab_status dab_binarize_train(const float* d_W, int64_t rows, int32_t n, int64_t ld_W, float* d_Wc, int64_t ld_Wc,
                              float* d_Wt, int64_t ld_Wt, int32_t* d_K, float* d_alpha, float* d_beta,
                              uint32_t* d_mask, int32_t ld_mask, uint32_t* d_row_flags, void* stream);
dab_status dab_binarize_backward(const float* d_Wc, int64_t rows, int32_t n, int64_t ld_Wc, const uint32_t* d_mask,
                                 int32_t ld_mask, const int32_t* d_K, const float* d_grad_Wt, int64_t ld_grad_Wt,
                                 float* d_grad_W, int64_t ld_grad_W, void* stream);

/*
 * dab_binary_conv_host — the same layer for a caller whose tensors live in host memory.  The batch is cut into 2 to
 * 16 chunks of images (of at least 8 MB where the batch allows); host-to-device copies, the kernels (on `stream`) and device-to-host copies of successive
 * chunks overlap on three streams, and the call returns after everything has drained.  Use pinned host memory:
 * with pageable memory the copies are staged by the driver and do not overlap.  The two copy streams and a few
 * events are created on the first call on a device and kept for the life of the process (the only state the
 * library keeps besides dab_binary_conv_static's array); calls on one device are serialised by a lock.
 * The scratch must hold dab_binary_conv_host_workspace(desc) bytes (two input and two output chunk buffers plus
 * the conv scratch of one chunk).
 */
size_t dab_binary_conv_host_workspace(const dab_conv_desc* desc);
dab_status dab_binary_conv_host(const dab_conv_desc* desc, const float* h_x, const uint32_t* d_wmask, int32_t ldw,
                                const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* h_y,
                                void* d_workspace, size_t workspace_bytes, void* stream);

/*
 * dab_binary_conv_host_async — the same call without the final wait: it returns once all its copies and kernels
 * are queued, so that the next layer's copy-in overlaps this layer's last kernels and copy-out.  Unlike
 * dab_binary_conv_host, whose first copy waits for the work already queued on `stream`, this form starts copying
 * h_x at once: h_x must hold its data when the call is made (the filters, device data, are still read in stream
 * order).  h_y is complete,
 * and h_x, the filters and the workspace may be reused or freed, only after dab_binary_conv_host_wait (or a later
 * dab_binary_conv_host on the device) has returned.  A call whose workspace overlaps that of one of the last two
 * unfinished calls waits for it on the device, and at most two calls are left running at a time: give
 * consecutive layers two alternating workspaces to let them overlap.
 * dab_binary_conv_host_wait — blocks until every such call on the current device, and `stream`, have finished.
 */
dab_status dab_binary_conv_host_async(const dab_conv_desc* desc, const float* h_x, const uint32_t* d_wmask,
                                      int32_t ldw, const int32_t* d_wK, const float* d_walpha, const float* d_wbeta,
                                      float* h_y, void* d_workspace, size_t workspace_bytes, void* stream);
dab_status dab_binary_conv_host_wait(void* stream);

/*
 * dab_binary_conv_static — dab_binary_conv without a workspace argument.  The paper has no counterpart: this
 * entry point exists for callers that cannot allocate device memory themselves, for example code running
 * inside a plugin or callback interface that hands it device pointers for inputs and outputs only, or a
 * process whose memory pool is owned by another component and may not be grown after start-up.
 *
 * The scratch for the patch codes is a fixed array of DAB_STATIC_SCRATCH_BYTES in device global memory that
 * belongs to the library image: every GPU on which the library is used holds it until the process exits.
 * The call allocates and frees nothing.  A layer fits when dab_binary_conv_workspace(desc) is at most
 * dab_binary_conv_static_capacity(); larger layers are refused with DAB_ERR_UNSUPPORTED (use dab_binary_conv
 * with your own workspace, or split the batch).  Inputs, outputs and their meaning are those of
 * dab_binary_conv; the optional outputs are not available here.
 *
 * The first call on each device looks up the device address of the array (a synchronous runtime query made
 * with that device current); make that first call outside any stream capture.  All calls on a device share
 * the one array and it keeps whatever the last call left in it: nothing in it needs clearing because each call
 * overwrites all it reads, but two calls whose kernels can overlap on the GPU (different streams, no ordering
 * between them) race on it and must be serialised by the caller.
 */
#define DAB_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
size_t dab_binary_conv_static_capacity(void);
dab_status dab_binary_conv_static(const dab_conv_desc* desc, const float* d_x, const uint32_t* d_wmask, int32_t ldw,
                                  const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* d_y,
                                  void* stream);

/*
 * Whole networks (Section 5.1: Sketch-A-Net, ResNet-18 and GoogLeNet with "all but the first [and last] layer
 * binarized"; Appendix "Experimental details": no bias in the binarized layers).  A network is a HOST array of
 * dab_layer records run one after the other on a running tensor (NCHW fp32); a second, remembered tensor carries
 * the shortcut of a residual block.  The pointers inside a record are DEVICE pointers owned by the caller.
 *
 *   DAB_LAYER_CONV_DENSE   full-precision convolution: d_weights [Cout x C*kh*kw] fp32, d_bias Cout fp32 or NULL;
 *                          products summed in fp64 in element order (c, kh, kw), one rounding to fp32
 *   DAB_LAYER_CONV_BINARY  dab_binary_conv with the filters coded by dab_binarize (d_wmask, ldw, d_wK, d_walpha, d_wbeta)
 *   DAB_LAYER_AFFINE       y = d_scale[c] * x + d_shift[c] per channel, in fp64, one rounding (a folded normalisation)
 *   DAB_LAYER_RELU         y = x > 0 ? x : 0
 *   DAB_LAYER_MAXPOOL      maximum over the kh x kw window, positions outside the image skipped
 *   DAB_LAYER_SAVE         remember (a copy of) the running tensor
 *   DAB_LAYER_ADD          running tensor + remembered tensor (same shape), fp32
 * on_saved != 0 (CONV_DENSE, AFFINE, RELU, MAXPOOL): the layer transforms the remembered tensor instead of the
 * running one (the 1x1 projection of a shortcut).  Fully connected layers are convolutions whose kernel covers
 * their whole input.  Fields a kind does not use are ignored.
 *
 * dab_network_output_shape  shape of the running tensor after the last layer.
 * dab_network_workspace     bytes of scratch dab_network_forward needs (four tensors of the largest size in the chain
 *                           plus the scratch of its largest binarized layer); 0 if the chain is invalid.
 * dab_network_forward       queues every layer on `stream` and returns without synchronising.  d_y receives the
 *                           running tensor after the last layer.  h_layer_outputs (host array of `count` device
 *                           pointers, or NULL; entries may be NULL): where given, layer i writes its output there
 *                           instead of into the workspace, so that a caller can inspect every intermediate tensor.
 * DAB_ERR_INVALID_ARG for a chain that does not fit together (shapes, missing pointers, ADD without SAVE),
 * DAB_ERR_UNSUPPORTED for a binarized layer with C*kh*kw > DAB_MAX_N, DAB_ERR_WORKSPACE as elsewhere.
 */
typedef enum {
  DAB_LAYER_CONV_DENSE = 0, DAB_LAYER_CONV_BINARY = 1, DAB_LAYER_AFFINE = 2, DAB_LAYER_RELU = 3, DAB_LAYER_MAXPOOL = 4,
  DAB_LAYER_SAVE = 5, DAB_LAYER_ADD = 6
} dab_layer_kind;

typedef struct {
  int32_t kind;      /* dab_layer_kind */
  int32_t on_saved;
  int32_t Cout, kh, kw, stride_h, stride_w, pad_h, pad_w;
  int32_t ldw;
  const float* d_weights;
  const float* d_bias;
  const uint32_t* d_wmask;
  const int32_t* d_wK;
  const float* d_walpha;
  const float* d_wbeta;
  const float* d_scale;
  const float* d_shift;
} dab_layer;

dab_status dab_network_output_shape(const dab_layer* layers, int32_t count, int32_t N, int32_t C, int32_t H, int32_t W,
                                    int32_t* Cout, int32_t* Ho, int32_t* Wo);
size_t dab_network_workspace(const dab_layer* layers, int32_t count, int32_t N, int32_t C, int32_t H, int32_t W);
dab_status dab_network_forward(const dab_layer* layers, int32_t count, int32_t N, int32_t C, int32_t H, int32_t W,
                               const float* d_x, float* d_y, void* d_workspace, size_t workspace_bytes,
                               float* const* h_layer_outputs, void* stream);

/*
 * Which kernel forms the AND-popcounts of dab_binary_gemm and of every convolution entry point (Section 4.2
 * counts set bits with population-count instructions; an AND-popcount over n bits is also the dot product of
 * the two rows written as 0/1 bytes, which the tensor cores form exactly in 32-bit integers):
 *   DAB_CONTRACT_TENSOR  mask words are expanded to bytes in shared memory and multiplied by
 *                        tcgen05.mma kind::i8 into tensor memory;
 *   DAB_CONTRACT_POPC    AND, carry-save adders and population counts on the integer pipes;
 *   DAB_CONTRACT_AUTO    (default) the tensor-core kernel, except for problems so small (fewer 128 x 64
 *                        output tiles than the device has SMs) that its per-tile latency is all there is.
 * Both kernels give the same counts and the same outputs bit for bit.  The setting is process-wide and read at
 * each call; the two forced values exist so that the kernels can be tested and measured against each other.
 */
typedef enum { DAB_CONTRACT_AUTO = 0, DAB_CONTRACT_TENSOR = 1, DAB_CONTRACT_POPC = 2 } dab_contraction;
dab_status dab_set_contraction(dab_contraction path);
dab_contraction dab_get_contraction(void);

/*
 * Which kernels code the patches in dab_binarize_patches and the convolution entry points built on it, and the rows
 * in dab_binarize (Section 4.1 / Algorithm 1 per row; every choice gives the same codes bit for bit):
 *   DAB_PATCHES_SORT   every row is sorted in full (its exact zeros are only counted) and every split evaluated;
 *   DAB_PATCHES_PIXEL  patches of 257..8192 values: the values of every input pixel (its C channels) are counted once
 *                      per tile into buckets of power-of-two width, with exact fp64 sums; a patch adds the tables of
 *                      its kh*kw pixels, which gives the split size and prefix sum at every bucket edge exactly.  The
 *                      objective is convex in (split size, prefix sum), so inside a bucket it is bounded by its values
 *                      at the corners of the region the bucket's count, sum and value bounds allow; only the few
 *                      buckets whose bound reaches the best edge value are searched exactly.  Work per pixel is
 *                      shared by the up to kh*kw patches that contain it.  Patches it cannot settle (a hull of more
 *                      than 1024 values, a constant row without zeros, magnitudes outside 2^-40..2^40, a NaN or an
 *                      infinity in the tile) are sorted in full by a second kernel;
 *   DAB_PATCHES_HIST   rows and patches of 257..8192 values, one warp each: a histogram of the row's own values
 *                      quantised to 24 bits of its range, the same bound per bucket with a margin for the
 *                      quantisation, exact search of what survives; rows it cannot settle fall to the sorting kernel;
 *   DAB_PATCHES_AUTO   (default) patches: DAB_PATCHES_PIXEL wherever a patch spans several pixels and the layer has
 *                      at least 1024 patches; otherwise per tile of the input the sorting kernels for tiles with few non-zero values
 *                      and DAB_PATCHES_HIST for the others.  Rows of a matrix: DAB_PATCHES_HIST from 2048 rows on,
 *                      DAB_PATCHES_SORT below.
 * Process-wide, read once at the start of each call.
 */
typedef enum { DAB_PATCHES_AUTO = 0, DAB_PATCHES_SORT = 1, DAB_PATCHES_HIST = 2, DAB_PATCHES_PIXEL = 3 } dab_patch_coder;
dab_status dab_set_patch_coder(dab_patch_coder coder);
dab_patch_coder dab_get_patch_coder(void);

/*
 * The tensor-core kernel waits on hardware barriers with a time limit (about two seconds) instead of
 * forever; a wait that ran out is counted on the device and leaves that tile's outputs unwritten.
 * dab_contraction_wait_failures copies the current device's count since library load to *h_count (host
 * pointer).  Synchronises the device.  0 on every correct run.
 */
dab_status dab_contraction_wait_failures(uint32_t* h_count);

#ifdef __cplusplus
}
#endif
#endif

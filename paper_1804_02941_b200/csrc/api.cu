// C ABI of libdab: argument validation on the host, then launches.  No allocation, no global state.
#include "common.cuh"

using namespace dab;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline dab_status from_cuda(cudaError_t e) { return e == cudaSuccess ? DAB_OK : DAB_ERR_CUDA; }

constexpr size_t kAlign = 256;

struct ConvGeom {
  int32_t Ho, Wo, n, ld;
  int64_t patches;
};

bool conv_geom(const dab_conv_desc* d, ConvGeom* g) {
  if (!d) return false;
  if (d->N < 1 || d->C < 1 || d->H < 1 || d->W < 1 || d->Cout < 1 || d->kh < 1 || d->kw < 1) return false;
  if (d->stride_h < 1 || d->stride_w < 1 || d->pad_h < 0 || d->pad_w < 0) return false;
  int64_t eh = (int64_t)d->H + 2 * (int64_t)d->pad_h - d->kh, ew = (int64_t)d->W + 2 * (int64_t)d->pad_w - d->kw;
  if (eh < 0 || ew < 0) return false;
  int64_t n = (int64_t)d->C * d->kh * d->kw;
  if (n > DAB_MAX_N) return false;
  g->Ho = (int32_t)(eh / d->stride_h + 1);
  g->Wo = (int32_t)(ew / d->stride_w + 1);
  g->n = (int32_t)n;
  g->ld = dab_default_ld((int32_t)n);
  g->patches = (int64_t)d->N * g->Ho * g->Wo;
  return true;
}

struct ConvScratch {
  size_t off_K, off_gamma, off_delta, off_mask, total;
};

ConvScratch conv_scratch(const ConvGeom& g) {
  ConvScratch s;
  size_t P = (size_t)g.patches, o = 0;
  s.off_K = o;       o += round_up(P * sizeof(int32_t), kAlign);
  s.off_gamma = o;   o += round_up(P * sizeof(float), kAlign);
  s.off_delta = o;   o += round_up(P * sizeof(float), kAlign);
  s.off_mask = o;    o += round_up(P * (size_t)g.ld * sizeof(uint32_t), kAlign);
  s.total = o;
  return s;
}

}  // namespace

extern "C" {

const char* dab_status_string(dab_status s) {
  switch (s) {
    case DAB_OK: return "ok";
    case DAB_ERR_INVALID_ARG: return "invalid argument";
    case DAB_ERR_UNSUPPORTED: return "size beyond a supported limit";
    case DAB_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case DAB_ERR_CUDA: return "CUDA error";
  }
  return "unknown status";
}

int32_t dab_words_per_row(int32_t n) { return n < 1 ? 0 : (n + 31) / 32; }
int32_t dab_default_ld(int32_t n) { return (dab_words_per_row(n) + 3) / 4 * 4; }

dab_status dab_binarize(const float* d_values, int64_t rows, int32_t n, int64_t ld_values, int32_t* d_K,
                        float* d_alpha, float* d_beta, uint32_t* d_mask, int32_t ld_mask, uint32_t* d_row_flags,
                        void* stream) {
  if (rows < 0 || n < 1) return DAB_ERR_INVALID_ARG;
  if (n > DAB_MAX_N) return DAB_ERR_UNSUPPORTED;
  if (ld_values < n || ld_mask < dab_words_per_row(n) || (ld_mask & 3)) return DAB_ERR_INVALID_ARG;
  if (rows == 0) return DAB_OK;
  if (!d_values || !d_K || !d_alpha || !d_beta || !d_mask || !aligned16(d_mask)) return DAB_ERR_INVALID_ARG;
  return from_cuda(launch_binarize(d_values, rows, n, ld_values, d_K, d_alpha, d_beta, d_mask, ld_mask, d_row_flags,
                                   static_cast<cudaStream_t>(stream)));
}

dab_status dab_pack(const uint8_t* d_bits, int64_t rows, int32_t n, int64_t ld_bits, uint32_t* d_mask,
                    int32_t ld_mask, int32_t* d_K, void* stream) {
  if (rows < 0 || n < 1) return DAB_ERR_INVALID_ARG;
  if (n > DAB_MAX_N) return DAB_ERR_UNSUPPORTED;
  if (ld_bits < n || ld_mask < dab_words_per_row(n) || (ld_mask & 3)) return DAB_ERR_INVALID_ARG;
  if (rows == 0) return DAB_OK;
  if (!d_bits || !d_mask || !aligned16(d_mask)) return DAB_ERR_INVALID_ARG;
  return from_cuda(launch_pack(d_bits, rows, n, ld_bits, d_mask, ld_mask, d_K, static_cast<cudaStream_t>(stream)));
}

dab_status dab_binary_gemm(int64_t M, int64_t N, int32_t n, const uint32_t* d_A, int32_t lda, const int32_t* d_KA,
                           const float* d_gamma, const float* d_delta, const uint32_t* d_B, int32_t ldb,
                           const int32_t* d_KB, const float* d_alpha, const float* d_beta, float* d_C, int64_t ldc,
                           int32_t* d_p11, int64_t ldp, void* stream) {
  if (M < 0 || N < 0 || n < 1) return DAB_ERR_INVALID_ARG;
  if (n > DAB_MAX_N) return DAB_ERR_UNSUPPORTED;
  int32_t wd = dab_words_per_row(n);
  if (lda < wd || ldb < wd || (lda & 3) || (ldb & 3) || ldc < N) return DAB_ERR_INVALID_ARG;
  if (d_p11 && ldp < N) return DAB_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return DAB_OK;
  if (N > (int64_t)65535 * 64) return DAB_ERR_UNSUPPORTED;
  if (!d_A || !d_KA || !d_gamma || !d_delta || !d_B || !d_KB || !d_alpha || !d_beta || !d_C) return DAB_ERR_INVALID_ARG;
  if (!aligned16(d_A) || !aligned16(d_B)) return DAB_ERR_INVALID_ARG;
  GemmArgs g;
  g.M = M; g.N = N; g.n = n; g.words = (wd + 3) / 4 * 4;
  g.A = d_A; g.lda = lda; g.KA = d_KA; g.gamma = d_gamma; g.delta = d_delta;
  g.B = d_B; g.ldb = ldb; g.KB = d_KB; g.alpha = d_alpha; g.beta = d_beta;
  g.C = d_C;
  g.map.inner = M; g.map.outer_stride = 0; g.map.row_stride = ldc; g.map.col_stride = 1;
  g.p11 = d_p11; g.ldp = ldp;
  return from_cuda(launch_gemm(g, /*lanes_along_rows=*/false, static_cast<cudaStream_t>(stream)));
}

dab_status dab_conv_output_size(const dab_conv_desc* desc, int32_t* Ho, int32_t* Wo) {
  ConvGeom g;
  if (!Ho || !Wo || !conv_geom(desc, &g)) return DAB_ERR_INVALID_ARG;
  *Ho = g.Ho;
  *Wo = g.Wo;
  return DAB_OK;
}

size_t dab_binary_conv_workspace(const dab_conv_desc* desc) {
  ConvGeom g;
  if (!conv_geom(desc, &g)) return 0;
  return conv_scratch(g).total;
}

dab_status dab_binarize_patches(const dab_conv_desc* desc, const float* d_x, int32_t* d_pK, float* d_pgamma,
                                float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, void* stream) {
  if (!desc) return DAB_ERR_INVALID_ARG;
  if (desc->C > 0 && desc->kh > 0 && desc->kw > 0 && (int64_t)desc->C * desc->kh * desc->kw > DAB_MAX_N)
    return DAB_ERR_UNSUPPORTED;
  ConvGeom g;
  if (!conv_geom(desc, &g)) return DAB_ERR_INVALID_ARG;
  if (!d_x || !d_pK || !d_pgamma || !d_pdelta || !d_pmask) return DAB_ERR_INVALID_ARG;
  if (ldp < dab_words_per_row(g.n) || (ldp & 3) || !aligned16(d_pmask)) return DAB_ERR_INVALID_ARG;
  return from_cuda(launch_binarize_patches(*desc, g.Ho, g.Wo, d_x, d_pK, d_pgamma, d_pdelta, d_pmask, ldp, d_pflags,
                                           static_cast<cudaStream_t>(stream)));
}

dab_status dab_binary_conv_contract(const dab_conv_desc* desc, const uint32_t* d_pmask, int32_t ldp,
                                    const int32_t* d_pK, const float* d_pgamma, const float* d_pdelta,
                                    const uint32_t* d_wmask, int32_t ldw, const int32_t* d_wK, const float* d_walpha,
                                    const float* d_wbeta, float* d_y, int32_t* d_p11, void* stream) {
  ConvGeom g;
  if (!conv_geom(desc, &g)) return DAB_ERR_INVALID_ARG;
  if (!d_pmask || !d_pK || !d_pgamma || !d_pdelta || !d_wmask || !d_wK || !d_walpha || !d_wbeta || !d_y)
    return DAB_ERR_INVALID_ARG;
  int32_t wd = dab_words_per_row(g.n);
  if (ldp < wd || (ldp & 3) || !aligned16(d_pmask) || ldw < wd || (ldw & 3) || !aligned16(d_wmask))
    return DAB_ERR_INVALID_ARG;
  if (desc->Cout > 65535 * 64) return DAB_ERR_UNSUPPORTED;
  GemmArgs a;
  a.M = g.patches; a.N = desc->Cout; a.n = g.n; a.words = (wd + 3) / 4 * 4;
  a.A = d_pmask; a.lda = ldp; a.KA = d_pK; a.gamma = d_pgamma; a.delta = d_pdelta;
  a.B = d_wmask; a.ldb = ldw; a.KB = d_wK; a.alpha = d_walpha; a.beta = d_wbeta;
  a.C = d_y;
  int64_t HoWo = (int64_t)g.Ho * g.Wo;
  a.map.inner = HoWo; a.map.outer_stride = (int64_t)desc->Cout * HoWo; a.map.row_stride = 1; a.map.col_stride = HoWo;
  a.p11 = d_p11; a.ldp = desc->Cout;
  return from_cuda(launch_gemm(a, /*lanes_along_rows=*/true, static_cast<cudaStream_t>(stream)));
}

dab_status dab_binary_conv(const dab_conv_desc* desc, const float* d_x, const uint32_t* d_wmask, int32_t ldw,
                           const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* d_y,
                           void* d_workspace, size_t workspace_bytes, int32_t* d_pK, float* d_pgamma,
                           float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, int32_t* d_p11,
                           void* stream) {
  if (!desc) return DAB_ERR_INVALID_ARG;
  if (desc->C > 0 && desc->kh > 0 && desc->kw > 0 && (int64_t)desc->C * desc->kh * desc->kw > DAB_MAX_N)
    return DAB_ERR_UNSUPPORTED;
  ConvGeom g;
  if (!conv_geom(desc, &g)) return DAB_ERR_INVALID_ARG;
  if (!d_x || !d_wmask || !d_wK || !d_walpha || !d_wbeta || !d_y) return DAB_ERR_INVALID_ARG;
  if (d_pmask && (ldp < dab_words_per_row(g.n) || (ldp & 3) || !aligned16(d_pmask))) return DAB_ERR_INVALID_ARG;
  ConvScratch sc = conv_scratch(g);
  if (!d_workspace || (reinterpret_cast<uintptr_t>(d_workspace) % kAlign) || workspace_bytes < sc.total)
    return DAB_ERR_WORKSPACE;
  char* ws = static_cast<char*>(d_workspace);
  int32_t* pK = d_pK ? d_pK : reinterpret_cast<int32_t*>(ws + sc.off_K);
  float* pg = d_pgamma ? d_pgamma : reinterpret_cast<float*>(ws + sc.off_gamma);
  float* pd = d_pdelta ? d_pdelta : reinterpret_cast<float*>(ws + sc.off_delta);
  uint32_t* pm = d_pmask ? d_pmask : reinterpret_cast<uint32_t*>(ws + sc.off_mask);
  int32_t ldm = d_pmask ? ldp : g.ld;
  dab_status s = dab_binarize_patches(desc, d_x, pK, pg, pd, pm, ldm, d_pflags, stream);
  if (s != DAB_OK) return s;
  return dab_binary_conv_contract(desc, pm, ldm, pK, pg, pd, d_wmask, ldw, d_wK, d_walpha, d_wbeta, d_y, d_p11, stream);
}

size_t dab_binary_conv_host_workspace(const dab_conv_desc* desc) {
  ConvGeom g;
  if (!conv_geom(desc, &g)) return 0;
  size_t xb = round_up((size_t)desc->N * desc->C * desc->H * desc->W * sizeof(float), kAlign);
  size_t yb = round_up((size_t)g.patches * desc->Cout * sizeof(float), kAlign);
  return xb + yb + conv_scratch(g).total;
}

dab_status dab_binary_conv_host(const dab_conv_desc* desc, const float* h_x, const uint32_t* d_wmask, int32_t ldw,
                                const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* h_y,
                                void* d_workspace, size_t workspace_bytes, void* stream) {
  ConvGeom g;
  if (!conv_geom(desc, &g)) return DAB_ERR_INVALID_ARG;
  if (!h_x || !h_y) return DAB_ERR_INVALID_ARG;
  size_t need = dab_binary_conv_host_workspace(desc);
  if (!d_workspace || (reinterpret_cast<uintptr_t>(d_workspace) % kAlign) || workspace_bytes < need)
    return DAB_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  size_t x_bytes = (size_t)desc->N * desc->C * desc->H * desc->W * sizeof(float);
  size_t y_bytes = (size_t)g.patches * desc->Cout * sizeof(float);
  size_t xb = round_up(x_bytes, kAlign), yb = round_up(y_bytes, kAlign);
  char* ws = static_cast<char*>(d_workspace);
  float* d_x = reinterpret_cast<float*>(ws);
  float* d_y = reinterpret_cast<float*>(ws + xb);
  if (cudaMemcpyAsync(d_x, h_x, x_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return DAB_ERR_CUDA;
  dab_status s = dab_binary_conv(desc, d_x, d_wmask, ldw, d_wK, d_walpha, d_wbeta, d_y, ws + xb + yb,
                                 workspace_bytes - xb - yb, nullptr, nullptr, nullptr, nullptr, 0, nullptr, nullptr,
                                 stream);
  if (s != DAB_OK) return s;
  if (cudaMemcpyAsync(h_y, d_y, y_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DAB_ERR_CUDA;
  return from_cuda(cudaStreamSynchronize(st));
}

dab_status dab_popc_probe(uint32_t* d_sink, int32_t blocks, int32_t iters, void* stream) {
  if (!d_sink || blocks < 1 || iters < 0) return DAB_ERR_INVALID_ARG;
  return from_cuda(launch_popc_probe(d_sink, blocks, iters, static_cast<cudaStream_t>(stream)));
}

}  // extern "C"

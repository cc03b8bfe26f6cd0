// C ABI of libdab: argument validation on the host, then launches.  No device memory is allocated; the state the
// library keeps is listed in include/dab.h.
#include <atomic>
#include <mutex>

#include "common.cuh"

using namespace dab;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline dab_status from_cuda(cudaError_t e) { return e == cudaSuccess ? DAB_OK : DAB_ERR_CUDA; }

constexpr size_t kAlign = 256;

std::atomic<int> g_contraction{(int)DAB_CONTRACT_AUTO};

// The contraction kernel the process-wide setting names.  The tensor-core kernel tiles the column side
// (weights when lanes_along_rows, activations otherwise) at least 64 rows per grid row; a launch too tall for
// that takes the population-count kernel, and so does, under DAB_CONTRACT_AUTO, one with fewer 128 x 64 tiles
// than a B200 has SMs: there the tensor-core kernel is a chain of dependent stage rounds on a few SMs.
cudaError_t contract(const GemmArgs& g, bool lanes_along_rows, cudaStream_t stream) {
  const int64_t lane_rows = lanes_along_rows ? g.M : g.N, column_rows = lanes_along_rows ? g.N : g.M;
  const int mode = g_contraction.load(std::memory_order_relaxed);
  bool tensor = mode != (int)DAB_CONTRACT_POPC && column_rows <= (int64_t)65535 * 64;
  if (mode == (int)DAB_CONTRACT_AUTO && ((lane_rows + 127) / 128) * ((column_rows + 63) / 64) < sm_count()) tensor = false;
  return tensor ? launch_gemm_mma(g, lanes_along_rows, stream) : launch_gemm(g, lanes_along_rows, stream);
}

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
  g.c_extent = (M - 1) * ldc + N;
  g.p11 = d_p11; g.ldp = ldp;
  return from_cuda(contract(g, /*lanes_along_rows=*/false, static_cast<cudaStream_t>(stream)));
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

static dab_status code_patches(bool sign, const dab_conv_desc* desc, const float* d_x, int32_t* d_pK, float* d_pgamma,
                               float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, void* stream) {
  if (!desc) return DAB_ERR_INVALID_ARG;
  if (desc->C > 0 && desc->kh > 0 && desc->kw > 0 && (int64_t)desc->C * desc->kh * desc->kw > DAB_MAX_N)
    return DAB_ERR_UNSUPPORTED;
  ConvGeom g;
  if (!conv_geom(desc, &g)) return DAB_ERR_INVALID_ARG;
  if (!d_x || !d_pK || !d_pgamma || !d_pdelta || !d_pmask) return DAB_ERR_INVALID_ARG;
  if (ldp < dab_words_per_row(g.n) || (ldp & 3) || !aligned16(d_pmask)) return DAB_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return from_cuda(sign ? launch_sign_patches(*desc, g.Ho, g.Wo, d_x, d_pK, d_pgamma, d_pdelta, d_pmask, ldp, d_pflags, st)
                        : launch_binarize_patches(*desc, g.Ho, g.Wo, d_x, d_pK, d_pgamma, d_pdelta, d_pmask, ldp,
                                                  d_pflags, st));
}

dab_status dab_binarize_patches(const dab_conv_desc* desc, const float* d_x, int32_t* d_pK, float* d_pgamma,
                                float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, void* stream) {
  return code_patches(false, desc, d_x, d_pK, d_pgamma, d_pdelta, d_pmask, ldp, d_pflags, stream);
}

dab_status dab_sign_patches(const dab_conv_desc* desc, const float* d_x, int32_t* d_pK, float* d_pgamma,
                            float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, void* stream) {
  return code_patches(true, desc, d_x, d_pK, d_pgamma, d_pdelta, d_pmask, ldp, d_pflags, stream);
}

dab_status dab_sign_binarize(const float* d_values, int64_t rows, int32_t n, int64_t ld_values, int32_t* d_K,
                             float* d_alpha, float* d_beta, uint32_t* d_mask, int32_t ld_mask, uint32_t* d_row_flags,
                             void* stream) {
  if (rows < 0 || n < 1) return DAB_ERR_INVALID_ARG;
  if (n > DAB_MAX_N) return DAB_ERR_UNSUPPORTED;
  if (ld_values < n || ld_mask < dab_words_per_row(n) || (ld_mask & 3)) return DAB_ERR_INVALID_ARG;
  if (rows == 0) return DAB_OK;
  if (!d_values || !d_K || !d_alpha || !d_beta || !d_mask || !aligned16(d_mask)) return DAB_ERR_INVALID_ARG;
  return from_cuda(launch_sign_rows(d_values, rows, n, ld_values, d_K, d_alpha, d_beta, d_mask, ld_mask, d_row_flags,
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
  a.c_extent = (int64_t)desc->N * desc->Cout * HoWo;
  a.p11 = d_p11; a.ldp = desc->Cout;
  return from_cuda(contract(a, /*lanes_along_rows=*/true, static_cast<cudaStream_t>(stream)));
}

static dab_status conv_with_coder(bool sign, const dab_conv_desc* desc, const float* d_x, const uint32_t* d_wmask, int32_t ldw,
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
  dab_status s = code_patches(sign, desc, d_x, pK, pg, pd, pm, ldm, d_pflags, stream);
  if (s != DAB_OK) return s;
  return dab_binary_conv_contract(desc, pm, ldm, pK, pg, pd, d_wmask, ldw, d_wK, d_walpha, d_wbeta, d_y, d_p11, stream);
}

dab_status dab_binary_conv(const dab_conv_desc* desc, const float* d_x, const uint32_t* d_wmask, int32_t ldw,
                           const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* d_y,
                           void* d_workspace, size_t workspace_bytes, int32_t* d_pK, float* d_pgamma,
                           float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, int32_t* d_p11,
                           void* stream) {
  return conv_with_coder(false, desc, d_x, d_wmask, ldw, d_wK, d_walpha, d_wbeta, d_y, d_workspace, workspace_bytes,
                         d_pK, d_pgamma, d_pdelta, d_pmask, ldp, d_pflags, d_p11, stream);
}

dab_status dab_binary_conv_sign(const dab_conv_desc* desc, const float* d_x, const uint32_t* d_wmask, int32_t ldw,
                                const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* d_y,
                                void* d_workspace, size_t workspace_bytes, int32_t* d_pK, float* d_pgamma,
                                float* d_pdelta, uint32_t* d_pmask, int32_t ldp, uint32_t* d_pflags, int32_t* d_p11,
                                void* stream) {
  return conv_with_coder(true, desc, d_x, d_wmask, ldw, d_wK, d_walpha, d_wbeta, d_y, d_workspace, workspace_bytes,
                         d_pK, d_pgamma, d_pdelta, d_pmask, ldp, d_pflags, d_p11, stream);
}

// ---------------------------------------------------------------------------------------------------------
// Host-buffer convolution: the batch is cut into chunks of images and pipelined over three streams
// (copy-in | compute | copy-out) with two device buffers per direction, so that PCIe traffic in both directions
// overlaps the kernels.  The two copy streams and the events are created once per device and kept.
// ---------------------------------------------------------------------------------------------------------
namespace {

constexpr int kHostChunks = 16;                    // chunks per call at most
constexpr size_t kHostChunkBytes = 32u << 20;      // and no smaller than this (of input or output, whichever is larger):
                                                   // every chunk costs a fixed few tens of microseconds of launches and events

struct HostPipe {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, in_done[2] = {}, comp_done[2] = {}, out_done[2] = {};
  // The last two calls that were left running (dab_binary_conv_host_async): their workspace ranges and the events
  // that mark the end of their kernels and of their copies out.  A new call waits for those whose workspace it touches.
  struct Tail {
    const char* lo = nullptr;
    const char* hi = nullptr;
    cudaEvent_t comp = nullptr, out = nullptr;
    bool live = false;
  } tail[2];
  int next_tail = 0;
};

std::mutex g_host_mutex;
HostPipe g_host_pipe[64];

cudaError_t host_pipe(HostPipe** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  HostPipe& p = g_host_pipe[dev];
  if (!p.ready) {
    if ((e = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking)) != cudaSuccess) return e;
    if ((e = cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking)) != cudaSuccess) return e;
    if ((e = cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming)) != cudaSuccess) return e;
    for (int b = 0; b < 2; ++b) {
      if ((e = cudaEventCreateWithFlags(&p.in_done[b], cudaEventDisableTiming)) != cudaSuccess) return e;
      if ((e = cudaEventCreateWithFlags(&p.comp_done[b], cudaEventDisableTiming)) != cudaSuccess) return e;
      if ((e = cudaEventCreateWithFlags(&p.out_done[b], cudaEventDisableTiming)) != cudaSuccess) return e;
      if ((e = cudaEventCreateWithFlags(&p.tail[b].comp, cudaEventDisableTiming)) != cudaSuccess) return e;
      if ((e = cudaEventCreateWithFlags(&p.tail[b].out, cudaEventDisableTiming)) != cudaSuccess) return e;
    }
    p.ready = true;
  }
  *out = &p;
  return cudaSuccess;
}

struct HostPlan {
  int32_t chunk_imgs, chunks;
  size_t x_chunk, y_chunk, scratch, total;  // bytes (x_chunk, y_chunk rounded up to kAlign)
  size_t x_img, y_img;                      // bytes per image
};

bool host_plan(const dab_conv_desc* desc, const ConvGeom& g, HostPlan* p) {
  p->x_img = (size_t)desc->C * desc->H * desc->W * sizeof(float);
  p->y_img = (size_t)desc->Cout * g.Ho * g.Wo * sizeof(float);
  const size_t img_bytes = p->x_img > p->y_img ? p->x_img : p->y_img;
  int64_t chunks = (int64_t)((img_bytes * (size_t)desc->N + kHostChunkBytes - 1) / kHostChunkBytes);
  if (chunks > kHostChunks) chunks = kHostChunks;
  if (chunks < 2) chunks = 2;                       // two at least, so that copies and kernels overlap at all
  if (chunks > desc->N) chunks = desc->N;
  p->chunk_imgs = (int32_t)((desc->N + chunks - 1) / chunks);
  p->chunks = (desc->N + p->chunk_imgs - 1) / p->chunk_imgs;
  p->x_chunk = round_up(p->x_img * p->chunk_imgs, kAlign);
  p->y_chunk = round_up(p->y_img * p->chunk_imgs, kAlign);
  dab_conv_desc d = *desc;
  d.N = p->chunk_imgs;
  ConvGeom gc;
  if (!conv_geom(&d, &gc)) return false;
  p->scratch = conv_scratch(gc).total;
  p->total = 2 * p->x_chunk + 2 * p->y_chunk + p->scratch;
  return true;
}

}  // namespace

size_t dab_binary_conv_host_workspace(const dab_conv_desc* desc) {
  ConvGeom g;
  HostPlan p;
  if (!conv_geom(desc, &g) || !host_plan(desc, g, &p)) return 0;
  return p.total;
}

static dab_status conv_host(bool drain, const dab_conv_desc* desc, const float* h_x, const uint32_t* d_wmask, int32_t ldw,
                            const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* h_y,
                            void* d_workspace, size_t workspace_bytes, void* stream) {
  ConvGeom g;
  HostPlan pl;
  if (!conv_geom(desc, &g) || !host_plan(desc, g, &pl)) return DAB_ERR_INVALID_ARG;
  if (!h_x || !h_y) return DAB_ERR_INVALID_ARG;
  if (!d_workspace || (reinterpret_cast<uintptr_t>(d_workspace) % kAlign) || workspace_bytes < pl.total)
    return DAB_ERR_WORKSPACE;
  std::lock_guard<std::mutex> lock(g_host_mutex);  // the copy streams and events are shared by all calls
  HostPipe* hp = nullptr;
  if (host_pipe(&hp) != cudaSuccess) return DAB_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(d_workspace);
  float* xbuf[2] = {reinterpret_cast<float*>(ws), reinterpret_cast<float*>(ws + pl.x_chunk)};
  float* ybuf[2] = {reinterpret_cast<float*>(ws + 2 * pl.x_chunk), reinterpret_cast<float*>(ws + 2 * pl.x_chunk + pl.y_chunk)};
  char* scratch = ws + 2 * pl.x_chunk + 2 * pl.y_chunk;

#define DAB_TRY(call) do { if ((call) != cudaSuccess) { cudaStreamSynchronize(hp->in); cudaStreamSynchronize(hp->out); \
                           cudaStreamSynchronize(st); return DAB_ERR_CUDA; } } while (0)
  if (drain) {  // work already queued on the caller's stream comes before the first copy
    DAB_TRY(cudaEventRecord(hp->start, st));
    DAB_TRY(cudaStreamWaitEvent(hp->in, hp->start, 0));
  }  // (the queued form reads h_x as it is at the time of the call, so that its copies overlap the kernels before it)
  // earlier calls still running on a workspace that overlaps this one (or about to lose their record) come first
  HostPipe::Tail& slot = hp->tail[hp->next_tail];
  for (int i = 0; i < 2; ++i) {
    HostPipe::Tail& t = hp->tail[i];
    if (!t.live) continue;
    const bool overlap = ws < t.hi && t.lo < ws + pl.total;
    if (overlap || &t == &slot) {
      DAB_TRY(cudaStreamWaitEvent(hp->in, t.comp, 0));
      DAB_TRY(cudaStreamWaitEvent(hp->in, t.out, 0));
      DAB_TRY(cudaStreamWaitEvent(st, t.comp, 0));
      DAB_TRY(cudaStreamWaitEvent(st, t.out, 0));
      if (&t == &slot) t.live = false;
    }
  }
  dab_status status = DAB_OK;
  for (int c = 0; c < pl.chunks; ++c) {
    const int b = c & 1;
    const int32_t img0 = c * pl.chunk_imgs;
    const int32_t imgs = desc->N - img0 < pl.chunk_imgs ? desc->N - img0 : pl.chunk_imgs;
    // copy-in: the x buffer is free once the chunk that used it two rounds ago has been computed
    if (c >= 2) DAB_TRY(cudaStreamWaitEvent(hp->in, hp->comp_done[b], 0));
    DAB_TRY(cudaMemcpyAsync(xbuf[b], reinterpret_cast<const char*>(h_x) + (size_t)img0 * pl.x_img, pl.x_img * imgs,
                            cudaMemcpyHostToDevice, hp->in));
    DAB_TRY(cudaEventRecord(hp->in_done[b], hp->in));
    // compute: needs the input, and the y buffer must have been copied out
    DAB_TRY(cudaStreamWaitEvent(st, hp->in_done[b], 0));
    if (c >= 2) DAB_TRY(cudaStreamWaitEvent(st, hp->out_done[b], 0));
    dab_conv_desc d = *desc;
    d.N = imgs;
    status = dab_binary_conv(&d, xbuf[b], d_wmask, ldw, d_wK, d_walpha, d_wbeta, ybuf[b], scratch, pl.scratch, nullptr,
                             nullptr, nullptr, nullptr, 0, nullptr, nullptr, stream);
    if (status != DAB_OK) break;
    DAB_TRY(cudaEventRecord(hp->comp_done[b], st));
    // copy-out
    DAB_TRY(cudaStreamWaitEvent(hp->out, hp->comp_done[b], 0));
    DAB_TRY(cudaMemcpyAsync(reinterpret_cast<char*>(h_y) + (size_t)img0 * pl.y_img, ybuf[b], pl.y_img * imgs,
                            cudaMemcpyDeviceToHost, hp->out));
    DAB_TRY(cudaEventRecord(hp->out_done[b], hp->out));
  }
  if (!drain && status == DAB_OK) {  // leave it running: remember what it occupies
    DAB_TRY(cudaEventRecord(slot.comp, st));
    DAB_TRY(cudaEventRecord(slot.out, hp->out));
    slot.lo = ws;
    slot.hi = ws + pl.total;
    slot.live = true;
    hp->next_tail ^= 1;
    return DAB_OK;
  }
#undef DAB_TRY
  cudaError_t e1 = cudaStreamSynchronize(hp->in), e2 = cudaStreamSynchronize(st), e3 = cudaStreamSynchronize(hp->out);
  hp->tail[0].live = hp->tail[1].live = false;  // the copy-out stream has drained: nothing is left running
  if (status != DAB_OK) return status;
  return (e1 == cudaSuccess && e2 == cudaSuccess && e3 == cudaSuccess) ? DAB_OK : DAB_ERR_CUDA;
}

dab_status dab_binary_conv_host(const dab_conv_desc* desc, const float* h_x, const uint32_t* d_wmask, int32_t ldw,
                                const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* h_y,
                                void* d_workspace, size_t workspace_bytes, void* stream) {
  return conv_host(true, desc, h_x, d_wmask, ldw, d_wK, d_walpha, d_wbeta, h_y, d_workspace, workspace_bytes, stream);
}

dab_status dab_binary_conv_host_async(const dab_conv_desc* desc, const float* h_x, const uint32_t* d_wmask, int32_t ldw,
                                      const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* h_y,
                                      void* d_workspace, size_t workspace_bytes, void* stream) {
  return conv_host(false, desc, h_x, d_wmask, ldw, d_wK, d_walpha, d_wbeta, h_y, d_workspace, workspace_bytes, stream);
}

dab_status dab_binary_conv_host_wait(void* stream) {
  std::lock_guard<std::mutex> lock(g_host_mutex);
  HostPipe* hp = nullptr;
  if (host_pipe(&hp) != cudaSuccess) return DAB_ERR_CUDA;
  cudaError_t e1 = cudaStreamSynchronize(hp->in), e2 = cudaStreamSynchronize(static_cast<cudaStream_t>(stream)),
              e3 = cudaStreamSynchronize(hp->out);
  hp->tail[0].live = hp->tail[1].live = false;
  return (e1 == cudaSuccess && e2 == cudaSuccess && e3 == cudaSuccess) ? DAB_OK : DAB_ERR_CUDA;
}

dab_status dab_set_contraction(dab_contraction path) {
  if (path != DAB_CONTRACT_AUTO && path != DAB_CONTRACT_TENSOR && path != DAB_CONTRACT_POPC) return DAB_ERR_INVALID_ARG;
  g_contraction.store((int)path, std::memory_order_relaxed);
  return DAB_OK;
}

dab_status dab_set_patch_coder(dab_patch_coder coder) {
  if (coder != DAB_PATCHES_AUTO && coder != DAB_PATCHES_SORT && coder != DAB_PATCHES_HIST && coder != DAB_PATCHES_PIXEL)
    return DAB_ERR_INVALID_ARG;
  set_patch_coder_mode((int)coder);
  return DAB_OK;
}

dab_patch_coder dab_get_patch_coder(void) { return (dab_patch_coder)patch_coder_mode(); }

dab_contraction dab_get_contraction(void) { return (dab_contraction)g_contraction.load(std::memory_order_relaxed); }

dab_status dab_contraction_wait_failures(uint32_t* h_count) {
  if (!h_count) return DAB_ERR_INVALID_ARG;
  unsigned int c = 0, w = 0;
  cudaError_t e = read_mma_wait_timeouts(&c);
  if (e == cudaSuccess) e = read_wbin_wait_timeouts(&w);
  *h_count = c + w;
  return from_cuda(e);
}

size_t dab_wbin_conv_workspace(const dab_conv_desc* desc) {
  ConvGeom g;
  if (!conv_geom(desc, &g)) return 0;
  return round_up((size_t)desc->N * desc->H * desc->W * sizeof(uint32_t), kAlign);
}

dab_status dab_wbin_conv(const dab_conv_desc* desc, const float* d_x, const uint32_t* d_wmask, int32_t ldw,
                         const float* d_walpha, const float* d_wbeta, float* d_y, void* d_workspace,
                         size_t workspace_bytes, void* stream) {
  if (!desc) return DAB_ERR_INVALID_ARG;
  if (desc->C > 0 && desc->kh > 0 && desc->kw > 0 && (int64_t)desc->C * desc->kh * desc->kw > DAB_MAX_N)
    return DAB_ERR_UNSUPPORTED;
  ConvGeom g;
  if (!conv_geom(desc, &g)) return DAB_ERR_INVALID_ARG;
  if (!d_x || !d_wmask || !d_walpha || !d_wbeta || !d_y) return DAB_ERR_INVALID_ARG;
  if (ldw < dab_words_per_row(g.n) || (ldw & 3) || !aligned16(d_wmask)) return DAB_ERR_INVALID_ARG;
  if (desc->Cout > 65535 * 64 || (int64_t)desc->C * desc->H * desc->W > 0x7FFFFFFF) return DAB_ERR_UNSUPPORTED;
  if ((int64_t)desc->N * desc->H * desc->W > (int64_t)0x7FFFFFFF * 256) return DAB_ERR_UNSUPPORTED;
  if (!d_workspace || (reinterpret_cast<uintptr_t>(d_workspace) % kAlign) ||
      workspace_bytes < dab_wbin_conv_workspace(desc))
    return DAB_ERR_WORKSPACE;
  cudaError_t e = launch_wbin_conv(*desc, g.Ho, g.Wo, d_x, d_wmask, ldw, d_walpha, d_wbeta, d_y,
                                   static_cast<uint32_t*>(d_workspace), static_cast<cudaStream_t>(stream));
  if (e == cudaErrorInvalidValue) return DAB_ERR_UNSUPPORTED;  // no tile of this layer fits shared memory
  return from_cuda(e);
}

dab_status dab_binarize_train(const float* d_W, int64_t rows, int32_t n, int64_t ld_W, float* d_Wc, int64_t ld_Wc,
                              float* d_Wt, int64_t ld_Wt, int32_t* d_K, float* d_alpha, float* d_beta,
                              uint32_t* d_mask, int32_t ld_mask, uint32_t* d_row_flags, void* stream) {
  if (rows < 0 || n < 1) return DAB_ERR_INVALID_ARG;
  if (n > DAB_MAX_N) return DAB_ERR_UNSUPPORTED;
  if (ld_W < n || ld_Wc < n || (d_Wt && ld_Wt < n) || ld_mask < dab_words_per_row(n) || (ld_mask & 3))
    return DAB_ERR_INVALID_ARG;
  if (rows == 0) return DAB_OK;
  if (!d_W || !d_Wc || !d_K || !d_alpha || !d_beta || !d_mask || !aligned16(d_mask)) return DAB_ERR_INVALID_ARG;
  return from_cuda(launch_train_forward(d_W, rows, n, ld_W, d_Wc, ld_Wc, d_Wt, ld_Wt, d_K, d_alpha, d_beta, d_mask,
                                        ld_mask, d_row_flags, static_cast<cudaStream_t>(stream)));
}

dab_status dab_binarize_backward(const float* d_Wc, int64_t rows, int32_t n, int64_t ld_Wc, const uint32_t* d_mask,
                                 int32_t ld_mask, const int32_t* d_K, const float* d_grad_Wt, int64_t ld_grad_Wt,
                                 float* d_grad_W, int64_t ld_grad_W, void* stream) {
  if (rows < 0 || n < 1) return DAB_ERR_INVALID_ARG;
  if (n > DAB_MAX_N) return DAB_ERR_UNSUPPORTED;
  if (ld_Wc < n || ld_grad_Wt < n || ld_grad_W < n || ld_mask < dab_words_per_row(n) || (ld_mask & 3))
    return DAB_ERR_INVALID_ARG;
  if (rows == 0) return DAB_OK;
  if (!d_Wc || !d_mask || !d_K || !d_grad_Wt || !d_grad_W) return DAB_ERR_INVALID_ARG;
  return from_cuda(launch_train_backward(d_Wc, ld_Wc, d_mask, ld_mask, d_K, rows, n, d_grad_Wt, ld_grad_Wt, d_grad_W,
                                         ld_grad_W, static_cast<cudaStream_t>(stream)));
}


}  // extern "C"

// Shared device helpers and internal launch declarations of libdab (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "dab.h"

// Checked indexing.  A build with -DDAB_DEBUG_BOUNDS compares every global-memory index its kernels form with the
// extent of the array it addresses.  The first violation seen by the kernels of a translation unit is recorded
// (source file as a hash of its name, line, index, extent) together with a count of all of them; a violating
// store is skipped and a violating load reads element 0 instead.  dab_debug_bounds_report() collects the records.
// In the ordinary build the two macros cost nothing: DAB_IN_BOUNDS is `true` and DAB_IDX is its first argument.
#ifdef DAB_DEBUG_BOUNDS
namespace dab {
namespace dbg {

struct Record {
  unsigned long long count;  // violations since the last reset
  long long index, extent;   // of the first one
  unsigned int file, line;   // FNV-1a hash of the base name of its source file, and its line
};

__host__ __device__ constexpr unsigned int file_id(const char* path) {
  const char* base = path;
  for (const char* p = path; *p; ++p)
    if (*p == '/') base = p + 1;
  unsigned int h = 2166136261u;
  for (const char* p = base; *p; ++p) h = (h ^ (unsigned char)*p) * 16777619u;
  return h;
}

static __device__ Record tu_record;

__device__ __forceinline__ bool in_bounds(long long index, long long extent, unsigned int file, unsigned int line) {
  if (index >= 0 && index < extent) return true;
  if (atomicAdd(&tu_record.count, 1ull) == 0ull) {
    tu_record.index = index;
    tu_record.extent = extent;
    tu_record.file = file;
    tu_record.line = line;
  }
  return false;
}

using Reader = cudaError_t (*)(Record* out, bool reset);
void register_reader(Reader reader);  // device.cu

static cudaError_t read_tu_record(Record* out, bool reset) {
  cudaError_t e = cudaMemcpyFromSymbol(out, tu_record, sizeof(Record));
  if (e == cudaSuccess && reset) {
    const Record zero{};
    e = cudaMemcpyToSymbol(tu_record, &zero, sizeof(Record));
  }
  return e;
}
static const bool tu_reader_registered = (register_reader(&read_tu_record), true);

}  // namespace dbg
}  // namespace dab
#define DAB_IN_BOUNDS(index, extent)                                                                    \
  ::dab::dbg::in_bounds((long long)(index), (long long)(extent),                                       \
                        std::integral_constant<unsigned int, ::dab::dbg::file_id(__FILE__)>::value, __LINE__)
#define DAB_IDX(index, extent) (DAB_IN_BOUNDS(index, extent) ? (index) : 0)
#else
#define DAB_IN_BOUNDS(index, extent) (true)
#define DAB_IDX(index, extent) (index)
#endif

namespace dab {

constexpr uint32_t kPadKey = 0xFFFFFFFFu;

// Monotone map fp32 -> uint32: a < b  <=>  key(a) < key(b); -0.0 and +0.0 share one key (x + 0.0f turns
// -0.0 into +0.0 and changes nothing else).
__device__ __forceinline__ uint32_t order_key(float x) {
  uint32_t b = __float_as_uint(__fadd_rn(x, 0.0f));
  return b ^ ((uint32_t)((int32_t)b >> 31) | 0x80000000u);
}

// Keys of non-finite values: +Inf/NaN(+) map to >= 0xFF800000, -Inf/NaN(-) to <= 0x007FFFFF.
__device__ __forceinline__ bool key_range_nonfinite(uint32_t kmin, uint32_t kmax) {
  return kmax >= 0xFF800000u || kmin <= 0x007FFFFFu;
}

__device__ __forceinline__ float key_value(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

__device__ __forceinline__ bool is_nonfinite(float x) {
  return (__float_as_uint(x) & 0x7F800000u) == 0x7F800000u;
}

// Objective of Algorithm 1 for a low partition of size s with sum P, row total T, row length n.
// Every operation rounds on its own (no fused multiply-add), in this order.
__device__ __forceinline__ double objective(double P, double T, int s, int n) {
  double Q = __dsub_rn(T, P);
  return __dadd_rn(__ddiv_rn(__dmul_rn(P, P), (double)s), __ddiv_rn(__dmul_rn(Q, Q), (double)(n - s)));
}

// Exact int32 -> fp64 without the conversion unit: 2^52 + 2^31 + p has p ^ 0x80000000 as its low word.
__device__ __forceinline__ double int_to_double(int p) {
  return __hiloint2double(0x43300000, (int)((unsigned)p ^ 0x80000000u)) - 4503601774854144.0;
}

// Four-term rescale in fp64, one rounding to fp32.  Term order is part of the contract.
__device__ __forceinline__ float rescale(int p11, int Ke, int Kf, int n, double a, double b, double g, double d) {
  int p10 = Ke - p11, p01 = Kf - p11, p00 = n - Ke - Kf + p11;
  double y = __dmul_rn(__dmul_rn(a, g), int_to_double(p11));
  y = __dadd_rn(y, __dmul_rn(__dmul_rn(a, d), int_to_double(p10)));
  y = __dadd_rn(y, __dmul_rn(__dmul_rn(b, g), int_to_double(p01)));
  y = __dadd_rn(y, __dmul_rn(__dmul_rn(b, d), int_to_double(p00)));
  return (float)y;
}

// Where an output element (row i of the activation side, column j of the weight side) is stored:
//   offset = (i / inner) * outer_stride + (i % inner) * row_stride + j * col_stride
// Row-major M x N: inner = M (never wraps), row_stride = ldc, col_stride = 1.
// NCHW conv output: inner = Ho*Wo, outer_stride = Cout*Ho*Wo, row_stride = 1, col_stride = Ho*Wo.
struct OutMap {
  int64_t inner, outer_stride, row_stride, col_stride;
};

struct GemmArgs {
  int64_t M, N;
  int32_t n, words;  // words = ceil(n/32) rounded up to a multiple of 4 (<= lda, ldb)
  const uint32_t* A;
  int32_t lda;
  const int32_t* KA;
  const float* gamma;
  const float* delta;
  const uint32_t* B;
  int32_t ldb;
  const int32_t* KB;
  const float* alpha;
  const float* beta;
  float* C;
  OutMap map;
  int64_t c_extent;  // elements from C to the end of the output it addresses (last offset of the map + 1)
  int32_t* p11;
  int64_t ldp;
};

// Number of SMs of the current device (read once per device).
int sm_count();
// Opts `kernel` in to `bytes` of dynamic shared memory on the current device unless an earlier call already did.
cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes);
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, size_t bytes) {
  return ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), bytes);
}

cudaError_t launch_binarize(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                            float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                            cudaStream_t stream);
cudaError_t launch_pack(const uint8_t* bits, int64_t rows, int32_t n, int64_t ld_bits, uint32_t* mask,
                        int32_t ld_mask, int32_t* K, cudaStream_t stream);
cudaError_t launch_gemm(const GemmArgs& args, bool lanes_along_rows, cudaStream_t stream);
// Tensor-core contraction; lanes_along_rows as for launch_gemm.  See gemm_mma.cu.
cudaError_t launch_gemm_mma(const GemmArgs& args, bool lanes_along_rows, cudaStream_t stream);
cudaError_t read_mma_wait_timeouts(unsigned int* count);
cudaError_t launch_binarize_patches(const dab_conv_desc& d, int32_t Ho, int32_t Wo, const float* x, int32_t* pK,
                                    float* pgamma, float* pdelta, uint32_t* pmask, int32_t ldp, uint32_t* pflags,
                                    cudaStream_t stream);
// Pixel-histogram patch coder (pixhist.cu): per-pixel bucket tables shared by the overlapping patches of a tile,
// then the full-sort kernel on the patches it marked.  *applicable = false: nothing was launched (no tile fits).
cudaError_t launch_binarize_patches_pixhist(const dab_conv_desc& d, int32_t Ho, int32_t Wo, const float* x,
                                            int32_t* pK, float* pgamma, float* pdelta, uint32_t* pmask, int32_t ldp,
                                            uint32_t* pflags, cudaStream_t stream, bool* applicable);
// Patch coder selection: 0 default, 1 sort-based only, 2 histogram-pruned per patch wherever it applies,
// 3 pixel-histogram coder wherever it applies.
int patch_coder_mode();
void set_patch_coder_mode(int mode);
constexpr int32_t kRowMark = -1;  // K of a row or of a tile's first patch that the next kernel of a chain has to code
cudaError_t launch_sign_rows(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K, float* alpha,
                             float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags, cudaStream_t stream);
cudaError_t launch_sign_patches(const dab_conv_desc& d, int32_t Ho, int32_t Wo, const float* x, int32_t* pK,
                                float* pgamma, float* pdelta, uint32_t* pmask, int32_t ldp, uint32_t* pflags,
                                cudaStream_t stream);
// Weights-only binarized convolution on the tensor cores; see wbin.cu.  pixmax: N*H*W words of scratch.
// cudaErrorInvalidValue: no tile fits.
cudaError_t launch_wbin_conv(const dab_conv_desc& d, int32_t Ho, int32_t Wo, const float* x, const uint32_t* wmask,
                             int32_t ldw, const float* walpha, const float* wbeta, float* y, uint32_t* pixmax,
                             cudaStream_t stream);
cudaError_t read_wbin_wait_timeouts(unsigned int* count);
// Training-side weight binarization and its gradient factor; see train.cu.  Wt may be null.
cudaError_t launch_train_forward(const float* W, int64_t rows, int32_t n, int64_t ld_W, float* Wc, int64_t ld_Wc,
                                 float* Wt, int64_t ld_Wt, int32_t* K, float* alpha, float* beta, uint32_t* mask,
                                 int32_t ld_mask, uint32_t* flags, cudaStream_t stream);
cudaError_t launch_train_backward(const float* Wc, int64_t ld_Wc, const uint32_t* mask, int32_t ld_mask,
                                  const int32_t* K, int64_t rows, int32_t n, const float* gWt, int64_t ld_g, float* gW,
                                  int64_t ld_gw, cudaStream_t stream);

}  // namespace dab

// dab_binary_conv_static: the binarized convolution for callers that cannot hand over device scratch memory.
//
// The patch codes that dab_binary_conv keeps in a caller-provided workspace live here in one fixed array
// in device global memory that is part of the library image.  Nothing is allocated or freed by this file.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = DAB_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Device-side storage.  In host code this name is only a handle for cudaGetSymbolAddress: it is not a device
// address and must never be passed to a kernel as it stands.
static __device__ __align__(256) unsigned char g_conv_scratch[kStaticScratchBytes];

std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};  // device address of g_conv_scratch on each device, once resolved

// Resolves (once per device, with that device current) the device address of the array.
dab_status scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DAB_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_conv_scratch);
    if (e != cudaSuccess || !p) return DAB_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return DAB_OK;
}

}  // namespace

extern "C" {

size_t dab_binary_conv_static_capacity(void) { return kStaticScratchBytes; }

dab_status dab_binary_conv_static(const dab_conv_desc* desc, const float* d_x, const uint32_t* d_wmask, int32_t ldw,
                                  const int32_t* d_wK, const float* d_walpha, const float* d_wbeta, float* d_y,
                                  void* stream) {
  if (!desc) return DAB_ERR_INVALID_ARG;
  if (desc->C > 0 && desc->kh > 0 && desc->kw > 0 && (int64_t)desc->C * desc->kh * desc->kw > DAB_MAX_N)
    return DAB_ERR_UNSUPPORTED;                            // row length beyond DAB_MAX_N, as dab_binary_conv reports it
  const size_t need = dab_binary_conv_workspace(desc);
  if (need == 0) return DAB_ERR_INVALID_ARG;               // impossible geometry
  if (need > kStaticScratchBytes) return DAB_ERR_UNSUPPORTED;  // layer too large for the built-in scratch
  void* scratch = nullptr;
  dab_status s = scratch_address(&scratch);
  if (s != DAB_OK) return s;
  // Every byte of the scratch that the contraction reads is written by the patch coder first (K, gamma, delta and
  // all ld words of every mask row), so nothing needs clearing between calls.
  return dab_binary_conv(desc, d_x, d_wmask, ldw, d_wK, d_walpha, d_wbeta, d_y, scratch, kStaticScratchBytes, nullptr,
                         nullptr, nullptr, nullptr, 0, nullptr, nullptr, stream);
}

}  // extern "C"

// Per-device facts and settings the launch code needs: the SM count (read once per device) and the opt-in to
// large dynamic shared memory of each kernel (raised only when a launch needs more than was set before).
// Both caches are guarded by one mutex; they hold nothing that a later call depends on for correctness.
#include <mutex>
#include <unordered_map>
#include <vector>

#include "common.cuh"
#include "dab_debug.h"

namespace dab {

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_mutex;
int g_sm_count[kMaxDevices] = {};
std::unordered_map<const void*, size_t> g_smem_set[kMaxDevices];
}  // namespace

int sm_count() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_sm_count[dev] == 0) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1) v = 148;
    g_sm_count[dev] = v;
  }
  return g_sm_count[dev];
}

cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  size_t& have = g_smem_set[dev][kernel];
  if (bytes <= have) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) have = bytes;
  return e;
}

}  // namespace dab

// Bounds report of the debug build: the per-translation-unit records of common.cuh, added up.
#ifdef DAB_DEBUG_BOUNDS
namespace dab {
namespace dbg {
namespace {
std::vector<Reader>& readers() {
  static std::vector<Reader> list;  // filled by static initialisers of the other translation units
  return list;
}
}  // namespace
void register_reader(Reader reader) { readers().push_back(reader); }
}  // namespace dbg
}  // namespace dab
#endif

extern "C" int32_t dab_debug_bounds_enabled(void) {
#ifdef DAB_DEBUG_BOUNDS
  return 1;
#else
  return 0;
#endif
}

extern "C" dab_status dab_debug_bounds_report(dab_bounds_report* h_report, int32_t reset) {
  if (h_report == nullptr) return DAB_ERR_INVALID_ARG;
  *h_report = dab_bounds_report{};
#ifdef DAB_DEBUG_BOUNDS
  if (cudaDeviceSynchronize() != cudaSuccess) return DAB_ERR_CUDA;
  for (dab::dbg::Reader read : dab::dbg::readers()) {
    dab::dbg::Record r;
    if (read(&r, reset != 0) != cudaSuccess) return DAB_ERR_CUDA;
    if (r.count != 0 && h_report->violations == 0) {
      h_report->index = r.index;
      h_report->extent = r.extent;
      h_report->file_hash = r.file;
      h_report->line = (int32_t)r.line;
    }
    h_report->violations += r.count;
  }
  return DAB_OK;
#else
  (void)reset;
  return DAB_ERR_UNSUPPORTED;
#endif
}

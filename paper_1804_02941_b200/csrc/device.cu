// Per-device facts and settings the launch code needs: the SM count (read once per device) and the opt-in to
// large dynamic shared memory of each kernel (raised only when a launch needs more than was set before).
// Both caches are guarded by one mutex; they hold nothing that a later call depends on for correctness.
#include <mutex>
#include <unordered_map>

#include "common.cuh"

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

// Test-only kernel: the bounded barrier wait of the tensor-core kernels (tc::mbar_wait) made to run out.
// One thread initialises an mbarrier that nothing ever arrives on and waits on it with a limit of a few
// thousand cycles; the wait must return false, set the caller's `dead` flag, bump the failure counter once per
// waiting thread, make later waits return at once, and the kernel must end.  No tensor-core instruction is used.
#include <cuda_runtime.h>
#include <stdint.h>

#include "tc.cuh"

__global__ void wait_timeout_kernel(long long limit, unsigned int* failures, int* out) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t bar_addr = dab::tc::smem_u32(&bar);
  if (threadIdx.x == 0) dab::tc::mbar_init(bar_addr, 1);
  __syncthreads();
  bool dead = false;
  const long long t0 = clock64();
  const bool first = dab::tc::mbar_wait(bar_addr, 0, dead, failures, limit);
  const long long waited = clock64() - t0;
  const bool second = dab::tc::mbar_wait(bar_addr, 0, dead, failures, limit);  // must not wait again
  __syncthreads();  // every thread still reaches the barriers that follow a failed wait
  if (threadIdx.x == 0) {
    out[0] = first ? 1 : 0;
    out[1] = second ? 1 : 0;
    out[2] = dead ? 1 : 0;
    out[3] = waited >= limit ? 1 : 0;
  }
}

extern "C" int run_wait_timeout(long long limit, int threads, unsigned int* d_failures, int* d_out) {
  wait_timeout_kernel<<<1, threads>>>(limit, d_failures, d_out);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return (int)e;
  return (int)cudaDeviceSynchronize();
}

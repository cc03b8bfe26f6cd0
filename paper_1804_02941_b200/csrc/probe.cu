// dab_popc_probe (include/dab_probe.h): a measurement aid for the population-count contraction kernel, kept out of
// the method's translation units.
#include "common.cuh"
#include "dab_probe.h"

namespace dab {

// Measurement aid: independent AND + POPC + IADD chains, 16 per thread per round.
__global__ void __launch_bounds__(256) popc_probe_kernel(uint32_t* sink, int iters) {
  uint32_t a[4], b[4];
  int acc[16];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    a[i] = 0x9E3779B9u * (threadIdx.x + 1 + i);
    b[i] = 0x85EBCA6Bu * (blockIdx.x + 7 + i);
  }
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = 0;
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i * 4 + j] += __popc(a[i] & b[j]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // change the operands so that nothing can be hoisted out of the loop
      a[i] = a[i] * 1664525u + 1013904223u;
      b[i] ^= a[i] >> 7;
    }
  }
  int s = 0;
#pragma unroll
  for (int i = 0; i < 16; ++i) s += acc[i];
  sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = (uint32_t)s;
}

static cudaError_t launch_popc_probe(uint32_t* sink, int32_t blocks, int32_t iters, cudaStream_t stream) {
  popc_probe_kernel<<<blocks, 256, 0, stream>>>(sink, iters);
  return cudaGetLastError();
}

}  // namespace dab

extern "C" dab_status dab_popc_probe(uint32_t* d_sink, int32_t blocks, int32_t iters, void* stream) {
  if (!d_sink || blocks < 1 || iters < 0) return DAB_ERR_INVALID_ARG;
  return dab::launch_popc_probe(d_sink, blocks, iters, static_cast<cudaStream_t>(stream)) == cudaSuccess ? DAB_OK : DAB_ERR_CUDA;
}

// dab_pack: 0/1 bytes -> packed 32-bit words.  HBM-bound: 1 byte read and 1 bit written per element.
#include "common.cuh"

namespace dab {

// Four bytes in one word -> 4 bits (bit k set iff byte k is non-zero).
__device__ __forceinline__ uint32_t nibble_of(uint32_t x) {
  uint32_t t = (((x & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | x) & 0x80808080u;  // bit 7 of each non-zero byte
  return (((t >> 7) * 0x00204081u) >> 21) & 0xFu;
}

// Fast path: rows start on 16-byte boundaries.  A thread turns 16 bytes into 16 bits; a lane pair makes a word.
__global__ void __launch_bounds__(256) pack_aligned_kernel(const uint8_t* __restrict__ bits, int64_t rows, int32_t n,
                                                           int64_t ld_bits, uint32_t* __restrict__ mask,
                                                           int32_t ld_mask, int32_t* __restrict__ K) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  const int64_t warp0 = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  const int64_t warp_stride = (int64_t)gridDim.x * warps_per_block;
  for (int64_t row = warp0; row < rows; row += warp_stride) {
    const uint8_t* b = bits + row * ld_bits;
    uint32_t* m = mask + row * (int64_t)ld_mask;
    int count = 0;
    // one pass of the warp covers 512 elements = 16 words
    for (int w0 = 0; w0 < ld_mask; w0 += 16) {
      int e0 = w0 * 32 + lane * 16;
      uint32_t half = 0;
      if (e0 + 16 <= n) {
        uint4 q = *reinterpret_cast<const uint4*>(b + e0);
        half = nibble_of(q.x) | (nibble_of(q.y) << 4) | (nibble_of(q.z) << 8) | (nibble_of(q.w) << 12);
      } else {
        for (int k = 0; k < 16; ++k)
          if (e0 + k < n && b[e0 + k]) half |= 1u << k;
      }
      uint32_t other = __shfl_down_sync(0xFFFFFFFFu, half, 1);
      uint32_t word = half | (other << 16);
      int w = w0 + (lane >> 1);
      if ((lane & 1) == 0 && w < ld_mask) {
        m[w] = word;
        count += __popc(word);
      }
    }
    if (K) {
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) count += __shfl_down_sync(0xFFFFFFFFu, count, off);
      if (lane == 0) K[row] = count;
    }
  }
}

// General path (any alignment): a warp ballots 32 bytes into one word.
__global__ void __launch_bounds__(256) pack_bytes_kernel(const uint8_t* __restrict__ bits, int64_t rows, int32_t n,
                                                         int64_t ld_bits, uint32_t* __restrict__ mask,
                                                         int32_t ld_mask, int32_t* __restrict__ K) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  const int64_t warp0 = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  const int64_t warp_stride = (int64_t)gridDim.x * warps_per_block;
  for (int64_t row = warp0; row < rows; row += warp_stride) {
    const uint8_t* b = bits + row * ld_bits;
    uint32_t* m = mask + row * (int64_t)ld_mask;
    int count = 0;
    for (int w = 0; w < ld_mask; ++w) {
      int i = w * 32 + lane;
      bool bit = i < n && b[i] != 0;
      uint32_t word = __ballot_sync(0xFFFFFFFFu, bit);
      if (lane == 0) m[w] = word;
      count += __popc(word);
    }
    if (K && lane == 0) K[row] = count;
  }
}

cudaError_t launch_pack(const uint8_t* bits, int64_t rows, int32_t n, int64_t ld_bits, uint32_t* mask,
                        int32_t ld_mask, int32_t* K, cudaStream_t stream) {
  const int threads = 256, wpb = threads / 32;
  int64_t blocks = (rows + wpb - 1) / wpb;
  if (blocks > 148 * 64) blocks = 148 * 64;
  bool aligned = (reinterpret_cast<uintptr_t>(bits) % 16 == 0) && (ld_bits % 16 == 0);
  if (aligned)
    pack_aligned_kernel<<<(unsigned)blocks, threads, 0, stream>>>(bits, rows, n, ld_bits, mask, ld_mask, K);
  else
    pack_bytes_kernel<<<(unsigned)blocks, threads, 0, stream>>>(bits, rows, n, ld_bits, mask, ld_mask, K);
  return cudaGetLastError();
}

}  // namespace dab

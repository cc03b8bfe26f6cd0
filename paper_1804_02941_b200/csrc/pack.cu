// dab_pack: 0/1 bytes -> packed 32-bit words.  HBM-bound: 1 byte read and 1 bit written per element.
#include "common.cuh"

namespace dab {

// Four bytes in one word -> 4 bits (bit k set iff byte k is non-zero).
__device__ __forceinline__ uint32_t nibble_of(uint32_t x) {
  // bit 7 of every non-zero byte: adding 0x7F to the low seven bits carries into bit 7 unless they are all 0
  const uint32_t t = (((x & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | x) & 0x80808080u;
  // bits 7, 15, 23, 31 -> bits 28..31: the partial products of this multiplier land on distinct bits (no carries)
  return (t * 0x00204081u) >> 28;
}

__device__ __forceinline__ uint32_t bits16_of(uint4 q) {
  return nibble_of(q.x) | (nibble_of(q.y) << 4) | (nibble_of(q.z) << 8) | (nibble_of(q.w) << 12);
}

// Fast path: rows start on 16-byte boundaries.  Work is laid out flat over (row, word): a thread turns 32 bytes
// into one word, so all lanes stay busy however short the rows are.  Pad words come out as 0.
// magic = floor(2^32 / ld_mask) gives the row of a flat index with one multiply and one correction.
__global__ void __launch_bounds__(256) pack_aligned_kernel(const uint8_t* __restrict__ bits, int64_t rows, int32_t n,
                                                           int64_t ld_bits, uint32_t* __restrict__ mask,
                                                           int32_t ld_mask, uint32_t magic, int64_t row_begin) {
  const uint32_t total = (uint32_t)rows * (uint32_t)ld_mask;  // the host keeps this below 2^31 per launch
  for (uint32_t t = blockIdx.x * blockDim.x + threadIdx.x; t < total; t += gridDim.x * blockDim.x) {
    uint32_t row = __umulhi(t, magic);
    uint32_t w = t - row * (uint32_t)ld_mask;
    if (w >= (uint32_t)ld_mask) { w -= ld_mask; ++row; }
    const int e0 = (int)w * 32;
    const int64_t bit_extent = (row_begin + rows - 1) * ld_bits + n;  // bytes up to the end of this launch's last row
    const int64_t b0 = (row_begin + row) * ld_bits + e0;
    const uint8_t* b = bits + b0;
    uint32_t word = 0;
    if (e0 + 32 <= n) {
      const uint4 q0 = __ldg(reinterpret_cast<const uint4*>(bits + DAB_IDX(b0, bit_extent - 15)));
      const uint4 q1 = __ldg(reinterpret_cast<const uint4*>(bits + DAB_IDX(b0 + 16, bit_extent - 15)));
      word = bits16_of(q0) | (bits16_of(q1) << 16);
    } else if (e0 < n) {  // the one ragged word of a row; words past the row stay 0
      for (int k = 0; k < n - e0; ++k)
        if (b[DAB_IDX(k, bit_extent - b0)]) word |= 1u << k;
    }
    if (DAB_IN_BOUNDS((row_begin + row) * (int64_t)ld_mask + w, (row_begin + rows) * (int64_t)ld_mask))
      mask[(row_begin + row) * (int64_t)ld_mask + w] = word;
  }
}

// Ones per row from the packed words (second, small pass over 1/8 byte per element): a thread per row for
// short rows (128-bit loads, every fetched sector fully used), a warp per row for long ones.
__global__ void __launch_bounds__(256) count_ones_thread_kernel(const uint32_t* __restrict__ mask, int64_t rows,
                                                                int32_t ld_mask, int32_t* __restrict__ K) {
  for (int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; row < rows; row += (int64_t)gridDim.x * blockDim.x) {
    const uint4* m = reinterpret_cast<const uint4*>(mask + row * (int64_t)ld_mask);
    int c = 0;
    for (int q = 0; q < ld_mask / 4; ++q) {
      const uint4 v = __ldg(m + DAB_IDX(q, ld_mask / 4));
      c += __popc(v.x) + __popc(v.y) + __popc(v.z) + __popc(v.w);
    }
    if (DAB_IN_BOUNDS(row, rows)) K[row] = c;
  }
}

__global__ void __launch_bounds__(256) count_ones_warp_kernel(const uint32_t* __restrict__ mask, int64_t rows,
                                                              int32_t ld_mask, int32_t* __restrict__ K) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t row = warp0; row < rows; row += nwarps) {
    int c = 0;
    for (int w = lane; w < ld_mask; w += 32) c += __popc(mask[DAB_IDX(row * (int64_t)ld_mask + w, rows * ld_mask)]);
    c = __reduce_add_sync(0xFFFFFFFFu, c);
    if (lane == 0 && DAB_IN_BOUNDS(row, rows)) K[row] = c;
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
      bool bit = i < n && b[DAB_IDX(i, n)] != 0;
      uint32_t word = __ballot_sync(0xFFFFFFFFu, bit);
      if (lane == 0 && DAB_IN_BOUNDS(row * ld_mask + w, rows * ld_mask)) m[w] = word;
      count += __popc(word);
    }
    if (K && lane == 0 && DAB_IN_BOUNDS(row, rows)) K[row] = count;
  }
}

cudaError_t launch_pack(const uint8_t* bits, int64_t rows, int32_t n, int64_t ld_bits, uint32_t* mask,
                        int32_t ld_mask, int32_t* K, cudaStream_t stream) {
  const int threads = 256, wpb = threads / 32;
  int64_t blocks = (rows + wpb - 1) / wpb;
  if (blocks > sm_count() * 64) blocks = sm_count() * 64;
  bool aligned = (reinterpret_cast<uintptr_t>(bits) % 16 == 0) && (ld_bits % 16 == 0);
  if (aligned) {
    const uint32_t magic = (uint32_t)(0x100000000ull / (uint64_t)ld_mask);  // ld_mask >= 4
    const int64_t rows_per_launch = (int64_t)0x7FFFFFFF / ld_mask;
    for (int64_t r0 = 0; r0 < rows; r0 += rows_per_launch) {
      const int64_t nr = rows - r0 < rows_per_launch ? rows - r0 : rows_per_launch;
      int64_t pb = (nr * ld_mask + threads - 1) / threads;
      if (pb > sm_count() * 32) pb = sm_count() * 32;
      pack_aligned_kernel<<<(unsigned)pb, threads, 0, stream>>>(bits, nr, n, ld_bits, mask, ld_mask, magic, r0);
    }
    if (K) {
      if (ld_mask <= 64) {
        int64_t cb = (rows + threads - 1) / threads;
        if (cb > sm_count() * 32) cb = sm_count() * 32;
        count_ones_thread_kernel<<<(unsigned)cb, threads, 0, stream>>>(mask, rows, ld_mask, K);
      } else {
        count_ones_warp_kernel<<<(unsigned)blocks, threads, 0, stream>>>(mask, rows, ld_mask, K);
      }
    }
  } else
    pack_bytes_kernel<<<(unsigned)blocks, threads, 0, stream>>>(bits, rows, n, ld_bits, mask, ld_mask, K);
  return cudaGetLastError();
}

}  // namespace dab

// dab_binarize: the row coder of rowcode.cuh applied to the rows of a matrix (one warp per row for up to 1024
// values, a group of 2..16 warps beyond).
#include "rowcode.cuh"

namespace dab {

// ---------------------------------------------------------------------------------------------------------
// Rows of a matrix, one warp per row (n <= 32*R).
// ---------------------------------------------------------------------------------------------------------
template <int R, bool kFull>
__global__ void __launch_bounds__(kWarpsPerCta * 32) binarize_rows_warp_kernel(
    const float* __restrict__ values, int64_t rows, int32_t n, int64_t ld_values, int32_t* __restrict__ K_out,
    float* __restrict__ alpha_out, float* __restrict__ beta_out, uint32_t* __restrict__ mask_out, int32_t ld_mask,
    uint32_t* __restrict__ flags_out) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* rcp = reinterpret_cast<double*>(smem_raw);
  uint32_t* scratch_all = reinterpret_cast<uint32_t*>(rcp + rcp_table_slots(n));
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* scratch = scratch_all + warp * (32 * R);
  fill_reciprocals(rcp, n, threadIdx.x, blockDim.x);
  __syncthreads();

  for (int64_t row = (int64_t)blockIdx.x * kWarpsPerCta + warp; row < rows; row += (int64_t)gridDim.x * kWarpsPerCta) {
    const float* v = values + row * ld_values;
    auto keyof = [v](int i) { return order_key(__ldg(v + i)); };
    uint32_t kreg[R];
    RowResult res = warp_code_row<R, kFull>(keyof, n, lane, scratch, rcp, kreg);
    if (lane == 0) {
      K_out[row] = res.K;
      alpha_out[row] = res.alpha;
      beta_out[row] = res.beta;
      if (flags_out) flags_out[row] = res.flags;
    }
    uint32_t mine = warp_mask_words<R, kFull>(kreg, n, lane, res);
    uint32_t* mrow = mask_out + row * (int64_t)ld_mask;
    for (int w = lane; w < ld_mask; w += 32) mrow[w] = (w < 32) ? mine : 0u;
  }
}

// ---------------------------------------------------------------------------------------------------------
// Rows of a matrix, a group of W > 1 warps per row.
// ---------------------------------------------------------------------------------------------------------
template <int W, int WARPS, int R, bool kFull, bool kTable>
__global__ void __launch_bounds__(WARPS * 32) binarize_rows_group_kernel(
    const float* __restrict__ values, int64_t rows, int32_t n, int64_t ld_values, int32_t* __restrict__ K_out,
    float* __restrict__ alpha_out, float* __restrict__ beta_out, uint32_t* __restrict__ mask_out, int32_t ld_mask,
    uint32_t* __restrict__ flags_out, int scratch_words) {
  constexpr int G = WARPS / W;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* rcp = reinterpret_cast<double*>(smem_raw);
  GroupShared* gs_all = reinterpret_cast<GroupShared*>(rcp + (kTable ? rcp_table_slots(n) : 0));
  uint32_t* scratch_all = reinterpret_cast<uint32_t*>(gs_all + G);

  const int group = threadIdx.x / (32 * W);
  const int tig = threadIdx.x % (32 * W);
  GroupShared* gs = gs_all + group;
  uint32_t* scratch = scratch_all + (size_t)group * scratch_words;
  const int bar_id = 1 + group;
  if (kTable) {
    fill_reciprocals(rcp, n, threadIdx.x, blockDim.x);
    __syncthreads();
  }

  for (int64_t row = (int64_t)blockIdx.x * G + group; row < rows; row += (int64_t)gridDim.x * G) {
    const float* v = values + row * ld_values;
    auto keyof = [v](int i) { return order_key(__ldg(v + i)); };
    uint32_t kreg[R];
    group_code_row<W, R, kFull, kTable>(keyof, n, tig, scratch, gs, bar_id, rcp, kreg);
    const RowResult res = gs->result;
    if (tig == 0) {
      K_out[row] = res.K;
      alpha_out[row] = res.alpha;
      beta_out[row] = res.beta;
      if (flags_out) flags_out[row] = res.flags;
    }
    group_store_mask<W, R, kFull>(kreg, n, ld_mask, tig, res, mask_out + row * (int64_t)ld_mask);
    group_barrier(bar_id, 32 * W);  // gs->result is overwritten by the next row
  }
}

template <int R, bool kFull>
static cudaError_t launch_rows_warp(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                                    float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                                    cudaStream_t stream) {
  auto kern = binarize_rows_warp_kernel<R, kFull>;
  size_t smem = sizeof(double) * rcp_table_slots(n) + sizeof(uint32_t) * 32 * R * kWarpsPerCta;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int64_t blocks = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
  if (blocks > 148 * 16) blocks = 148 * 16;
  kern<<<(unsigned)blocks, kWarpsPerCta * 32, smem, stream>>>(values, rows, n, ld_values, K, alpha, beta, mask,
                                                              ld_mask, flags);
  return cudaGetLastError();
}

template <int W, int WARPS, int R, bool kFull, bool kTable>
static cudaError_t launch_rows_group(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                                     float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                                     cudaStream_t stream) {
  constexpr int G = WARPS / W;
  auto kern = binarize_rows_group_kernel<W, WARPS, R, kFull, kTable>;
  int sw = scratch_words_for(n, W);
  size_t smem = (kTable ? sizeof(double) * rcp_table_slots(n) : 0) + sizeof(GroupShared) * G + sizeof(uint32_t) * (size_t)sw * G;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int64_t blocks = (rows + G - 1) / G;
  if (blocks > 148 * 16) blocks = 148 * 16;
  kern<<<(unsigned)blocks, WARPS * 32, smem, stream>>>(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask,
                                                       flags, sw);
  return cudaGetLastError();
}

cudaError_t launch_binarize(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                            float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                            cudaStream_t stream) {
#define DAB_ARGS values, rows, n, ld_values, K, alpha, beta, mask, ld_mask, flags, stream
  // A matrix may have few rows (a layer's filters), so a row gets enough warps for at most 8 keys per thread
  // even when none of its values is zero: short critical path per row, and the 8-key network is the most
  // efficient one per element.
  if (n <= 256) return launch_rows_warp<8, false>(DAB_ARGS);
  if (n <= 1024) return launch_rows_group<4, 8, 8, false, true>(DAB_ARGS);
  if (n <= 2048) return launch_rows_group<8, 8, 8, false, true>(DAB_ARGS);
  if (n <= 4096) return launch_rows_group<16, 16, 8, false, true>(DAB_ARGS);
  if (n <= 8192) return launch_rows_group<32, 32, 8, false, true>(DAB_ARGS);
  return launch_rows_group<32, 32, 16, false, false>(DAB_ARGS);
#undef DAB_ARGS
}

}  // namespace dab

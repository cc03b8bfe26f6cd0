// dab_binarize: the rows of a matrix through the sorting coder of rowcode.cuh (one warp per row for up to 256
// values, a group of 4..32 warps beyond) or, for large dense matrices, the histogram-pruned search of histcode.cuh.
#include "histcode.cuh"
#include "rowcode.cuh"

namespace dab {

// Whether any of the rows this CTA would take (row = (blockIdx.x + k * gridDim.x) * per_cta + g, g < per_cta) carries
// the mark of an earlier kernel of the call.  Every thread of the CTA gets the same answer.
__device__ __forceinline__ bool cta_has_marked_row(const int32_t* K_out, int64_t rows, int per_cta) {
  int any = 0;
  for (int64_t i = threadIdx.x;; i += blockDim.x) {
    const int64_t row = ((int64_t)blockIdx.x + (i / per_cta) * gridDim.x) * per_cta + i % per_cta;
    if (row >= rows) break;
    any |= K_out[DAB_IDX(row, rows)] == kRowMark;
  }
  return __syncthreads_or(any) != 0;
}

// ---------------------------------------------------------------------------------------------------------
// Rows of a matrix, one warp per row (n <= 32*R).
// ---------------------------------------------------------------------------------------------------------
template <int R, bool kFull>
__global__ void __launch_bounds__(kWarpsPerCta * 32) binarize_rows_warp_kernel(
    const float* __restrict__ values, int64_t rows, int32_t n, int64_t ld_values, int32_t* __restrict__ K_out,
    float* __restrict__ alpha_out, float* __restrict__ beta_out, uint32_t* __restrict__ mask_out, int32_t ld_mask,
    uint32_t* __restrict__ flags_out, int marked_only) {
  // marked_only: code only the rows an earlier kernel of the call marked (K = kRowMark); a CTA none of whose rows is
  // marked leaves at once
  if (marked_only && !cta_has_marked_row(K_out, rows, kWarpsPerCta)) return;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* rcp = reinterpret_cast<double*>(smem_raw);
  uint32_t* scratch_all = reinterpret_cast<uint32_t*>(rcp + rcp_table_slots(n));
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* scratch = scratch_all + warp * (32 * R);
  fill_reciprocals(rcp, n, threadIdx.x, blockDim.x);
  __syncthreads();

  for (int64_t row = (int64_t)blockIdx.x * kWarpsPerCta + warp; row < rows; row += (int64_t)gridDim.x * kWarpsPerCta) {
    if (marked_only && K_out[DAB_IDX(row, rows)] != kRowMark) continue;
    const float* v = values + row * ld_values;
    auto keyof = [v, n](int i) { return order_key(__ldg(v + DAB_IDX(i, n))); };
    uint32_t kreg[R];
    RowResult res = warp_code_row<R, kFull>(keyof, n, lane, scratch, rcp, kreg);
    if (lane == 0 && DAB_IN_BOUNDS(row, rows)) {
      K_out[row] = res.K;
      alpha_out[row] = res.alpha;
      beta_out[row] = res.beta;
      if (flags_out) flags_out[row] = res.flags;
    }
    uint32_t mine = warp_mask_words<R, kFull>(kreg, n, lane, res);
    uint32_t* mrow = mask_out + row * (int64_t)ld_mask;
    for (int w = lane; w < ld_mask; w += 32)
      if (DAB_IN_BOUNDS(row * ld_mask + w, rows * ld_mask)) mrow[w] = (w < 32) ? mine : 0u;
  }
}

// ---------------------------------------------------------------------------------------------------------
// Rows of a matrix, a group of W > 1 warps per row.
// ---------------------------------------------------------------------------------------------------------
template <int W, int WARPS, int R, bool kFull, bool kTable>
__global__ void __launch_bounds__(WARPS * 32) binarize_rows_group_kernel(
    const float* __restrict__ values, int64_t rows, int32_t n, int64_t ld_values, int32_t* __restrict__ K_out,
    float* __restrict__ alpha_out, float* __restrict__ beta_out, uint32_t* __restrict__ mask_out, int32_t ld_mask,
    uint32_t* __restrict__ flags_out, int scratch_words, int marked_only) {
  constexpr int G = WARPS / W;
  if (marked_only && !cta_has_marked_row(K_out, rows, G)) return;
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
    if (marked_only && K_out[DAB_IDX(row, rows)] != kRowMark) continue;  // the same for every thread of the group
    const float* v = values + row * ld_values;
    auto keyof = [v, n](int i) { return order_key(__ldg(v + DAB_IDX(i, n))); };
    uint32_t kreg[R];
    group_code_row<W, R, kFull, kTable>(keyof, n, tig, scratch, gs, bar_id, rcp, kreg);
    const RowResult res = gs->result;
    if (tig == 0 && DAB_IN_BOUNDS(row, rows)) {
      K_out[row] = res.K;
      alpha_out[row] = res.alpha;
      beta_out[row] = res.beta;
      if (flags_out) flags_out[row] = res.flags;
    }
    group_store_mask<W, R, kFull>(kreg, n, ld_mask, tig, res, mask_out, row, rows);
    group_barrier(bar_id, 32 * W);  // gs->result is overwritten by the next row
  }
}

template <int R, bool kFull>
static cudaError_t launch_rows_warp(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                                    float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                                    cudaStream_t stream, int marked_only) {
  auto kern = binarize_rows_warp_kernel<R, kFull>;
  size_t smem = sizeof(double) * rcp_table_slots(n) + sizeof(uint32_t) * 32 * R * kWarpsPerCta;
  cudaError_t e = ensure_dynamic_smem(kern, smem);
  if (e != cudaSuccess) return e;
  int64_t blocks = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
  if (blocks > sm_count() * 16) blocks = sm_count() * 16;
  kern<<<(unsigned)blocks, kWarpsPerCta * 32, smem, stream>>>(values, rows, n, ld_values, K, alpha, beta, mask,
                                                              ld_mask, flags, marked_only);
  return cudaGetLastError();
}

template <int W, int WARPS, int R, bool kFull, bool kTable>
static cudaError_t launch_rows_group(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                                     float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                                     cudaStream_t stream, int marked_only) {
  constexpr int G = WARPS / W;
  auto kern = binarize_rows_group_kernel<W, WARPS, R, kFull, kTable>;
  int sw = scratch_words_for(n, W);
  size_t smem = (kTable ? sizeof(double) * rcp_table_slots(n) : 0) + sizeof(GroupShared) * G + sizeof(uint32_t) * (size_t)sw * G;
  cudaError_t e = ensure_dynamic_smem(kern, smem);
  if (e != cudaSuccess) return e;
  int64_t blocks = (rows + G - 1) / G;
  if (blocks > sm_count() * 16) blocks = sm_count() * 16;
  kern<<<(unsigned)blocks, WARPS * 32, smem, stream>>>(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask,
                                                       flags, sw, marked_only);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------
// Rows of a matrix through the histogram-pruned search of histcode.cuh, one warp per row.  Four passes over the
// row (read through the caches): range of the non-zero values, histogram, gather of the hull, mask.  Rows it
// does not settle (a NaN or an infinity, a hull of more than 256 or 1024 values, too few non-zero values when
// min_density_pct is set) are marked with K = kRowMark for the sorting kernel that follows it on the stream.
// ---------------------------------------------------------------------------------------------------------
template <int BPL>
__global__ void __launch_bounds__(kWarpsPerCta * 32, 3) binarize_rows_hist_kernel(
    const float* __restrict__ values, int64_t rows, int32_t n, int64_t ld_values, int32_t* __restrict__ K_out,
    float* __restrict__ alpha_out, float* __restrict__ beta_out, uint32_t* __restrict__ mask_out, int32_t ld_mask,
    uint32_t* __restrict__ flags_out, int min_density_pct) {
  constexpr int B = 32 * BPL;
  constexpr int LOG2B = BPL == 1 ? 5 : BPL == 2 ? 6 : BPL == 4 ? 7 : 8;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* rcp = reinterpret_cast<double*>(smem_raw);
  int2* hist_all = reinterpret_cast<int2*>(rcp + rcp_table_slots(n));
  uint32_t* scratch_all = reinterpret_cast<uint32_t*>(hist_all + kWarpsPerCta * B);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int2* hist = hist_all + warp * B;
  uint32_t* scratch = scratch_all + warp * hist_cap(BPL);
  fill_reciprocals(rcp, n, threadIdx.x, blockDim.x);
  __syncthreads();
  const int qbits = quant_bits(n, LOG2B);
  const int rounds = (n + 31) >> 5;

  for (int64_t row = (int64_t)blockIdx.x * kWarpsPerCta + warp; row < rows; row += (int64_t)gridDim.x * kWarpsPerCta) {
    const float* v = values + row * ld_values;
    auto element = [v, n, lane](int k) {  // element of round k for this lane (+0.0 folds -0.0), 0.0 beyond the row
      const int i = k * 32 + lane;
      return i < n ? __fadd_rn(__ldg(v + DAB_IDX(i, n)), 0.0f) : 0.0f;
    };
    // pass 0: range and number of the non-zero values
    uint32_t kmin = kPadKey, kmax = 0u;
    int nz = 0;
#pragma unroll 4
    for (int k = 0; k < rounds; ++k) {
      const float x = element(k);
      if (x != 0.0f) {  // NaN compares unequal: counted, and seen as non-finite below
        const uint32_t key = order_key(x);
        kmin = min(kmin, key);
        kmax = max(kmax, key);
        ++nz;
      }
    }
    kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
    kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
    nz = __reduce_add_sync(0xFFFFFFFFu, nz);
    const bool any_nonzero = kmin <= kmax;
    bool retry = (any_nonzero && key_range_nonfinite(kmin, kmax)) || (int64_t)nz * 100 < (int64_t)min_density_pct * n;
    RowResult res;
    if (!retry) {
      const Quant qz = make_quant(any_nonzero ? key_value(kmin) : 0.0f, any_nonzero ? key_value(kmax) : 0.0f, qbits, LOG2B);
      auto sweep = [&](auto f) {
#pragma unroll 4
        for (int k = 0; k < rounds; ++k) f(element(k), k * 32 + lane < n);
      };
      retry = !hist_search<BPL>(sweep, n, qz, hist, scratch, rcp, lane, res);
    }
    if (retry) {
      if (lane == 0 && DAB_IN_BOUNDS(row, rows)) K_out[row] = kRowMark;
      continue;
    }
    if (lane == 0 && DAB_IN_BOUNDS(row, rows)) {
      K_out[row] = res.K;
      alpha_out[row] = res.alpha;
      beta_out[row] = res.beta;
      if (flags_out) flags_out[row] = res.flags;
    }
    const bool flip = res.mode == 1, none = res.mode == 2;
    const float tv = key_value(res.tkey);
    uint32_t* mrow = mask_out + row * (int64_t)ld_mask;
    const bool keep = !none;
    for (int kb = 0; kb < rounds; kb += 32) {  // 32 mask words at a time: word kb + j ends up in lane j
      const int kend = min(32, rounds - kb);
      uint32_t mine = 0;
#pragma unroll 4
      for (int kk = 0; kk < kend; ++kk) {
        const float x = element(kb + kk);
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, keep && ((kb + kk) * 32 + lane < n) && ((x >= tv) != flip));
        if (kk == lane) mine = word;
      }
      if (lane < kend && DAB_IN_BOUNDS(row * ld_mask + kb + lane, rows * ld_mask)) mrow[kb + lane] = mine;
    }
    for (int w = rounds + lane; w < ld_mask; w += 32)
      if (DAB_IN_BOUNDS(row * ld_mask + w, rows * ld_mask)) mrow[w] = 0u;
  }
}

template <int BPL>
static cudaError_t launch_rows_hist(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                                    float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                                    cudaStream_t stream, int min_density_pct) {
  auto kern = binarize_rows_hist_kernel<BPL>;
  size_t smem = sizeof(double) * rcp_table_slots(n) + (sizeof(int2) * 32 * BPL + sizeof(uint32_t) * hist_cap(BPL)) * kWarpsPerCta;
  cudaError_t e = ensure_dynamic_smem(kern, smem);
  if (e != cudaSuccess) return e;
  int64_t blocks = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
  if (blocks > sm_count() * 16) blocks = sm_count() * 16;
  kern<<<(unsigned)blocks, kWarpsPerCta * 32, smem, stream>>>(values, rows, n, ld_values, K, alpha, beta, mask,
                                                              ld_mask, flags, min_density_pct);
  return cudaGetLastError();
}

static cudaError_t launch_rows_sort(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                                    float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                                    cudaStream_t stream, int marked_only) {
#define DAB_ARGS values, rows, n, ld_values, K, alpha, beta, mask, ld_mask, flags, stream, marked_only
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

// Rows at which a matrix is large enough for one warp per row to fill the device: below it the sorting kernels,
// which put up to 32 warps on a row, finish sooner.
constexpr int64_t kHistMinRows = 2048;

cudaError_t launch_binarize(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                            float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                            cudaStream_t stream) {
  const int mode = patch_coder_mode();  // the setting covers the rows of matrices as well
  if (mode == 1 || n <= 256 || n > 8192 || (mode == 0 && rows < kHistMinRows))
    return launch_rows_sort(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask, flags, stream, 0);
  // The histogram-pruned search first; the sorting kernel then takes the rows it marked.
  cudaError_t e;
  const int min_density = 0;  // rows of any density: on matrices this large the search beats the sort on sparse rows too
  if (n < 1024) e = launch_rows_hist<2>(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask, flags, stream, min_density);
  else if (n < 4096) e = launch_rows_hist<4>(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask, flags, stream, min_density);
  else e = launch_rows_hist<8>(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask, flags, stream, min_density);
  if (e != cudaSuccess) return e;
  return launch_rows_sort(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask, flags, stream, 1);
}

}  // namespace dab

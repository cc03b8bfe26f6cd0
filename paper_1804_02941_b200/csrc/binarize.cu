// dab_binarize: one CTA per row.  Sort the row's order-preserving keys in shared memory, scan the
// sorted values in fp64, evaluate the objective of Algorithm 1 at every split between distinct
// values, reduce to the arg-max under the tie rule, then write K, alpha, beta and the packed mask.
#include "common.cuh"

namespace dab {

struct Best {
  double D;
  double P;
  int s;
};

__device__ __forceinline__ bool better(const Best& a, const Best& b) {  // is a preferred over b
  return a.D > b.D || (a.D == b.D && a.s > b.s);
}

__device__ __forceinline__ Best shfl_down_best(const Best& v, int off) {
  Best r;
  r.D = __shfl_down_sync(0xFFFFFFFFu, v.D, off);
  r.P = __shfl_down_sync(0xFFFFFFFFu, v.P, off);
  r.s = __shfl_down_sync(0xFFFFFFFFu, v.s, off);
  return r;
}

template <int NPAD, int THREADS>
__global__ void __launch_bounds__(THREADS) binarize_rows_kernel(const float* __restrict__ values, int64_t rows,
                                                                int32_t n, int64_t ld_values,
                                                                int32_t* __restrict__ K_out,
                                                                float* __restrict__ alpha_out,
                                                                float* __restrict__ beta_out,
                                                                uint32_t* __restrict__ mask_out, int32_t ld_mask,
                                                                uint32_t* __restrict__ flags_out) {
  constexpr int L = NPAD / THREADS;  // sorted positions owned by one thread in the scan
  constexpr int WARPS = THREADS / 32;
  static_assert(NPAD % THREADS == 0 && THREADS % 32 == 0, "shape");
  extern __shared__ uint32_t keys[];  // NPAD keys
  __shared__ double warp_sum[WARPS];
  __shared__ Best warp_best[WARPS];
  __shared__ uint32_t s_tkey;
  __shared__ int s_mode;  // 0: e = [w >= t], 1: e = [w < t], 2: empty mask

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    const float* v = values + row * ld_values;
    uint32_t* mrow = mask_out + row * (int64_t)ld_mask;

    int bad = 0;
    for (int i = tid; i < NPAD; i += THREADS) {
      uint32_t k = kPadKey;
      if (i < n) {
        float x = v[i];
        bad |= is_nonfinite(x);
        k = order_key(x);
      }
      keys[i] = k;
    }
    bad = __syncthreads_or(bad);

    if (!bad) {
      // Bitonic sort, ascending; the pad keys end up behind the n real ones.
      for (int k = 2; k <= NPAD; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
          for (int t = tid; t < NPAD / 2; t += THREADS) {
            int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
            int p = i | j;
            uint32_t a = keys[i], b = keys[p];
            bool up = (i & k) == 0;
            if ((a > b) == up) {
              keys[i] = b;
              keys[p] = a;
            }
          }
          __syncthreads();
        }
      }
    }

    const bool constant = !bad && keys[0] == keys[n - 1];

    if (!bad && !constant) {
      // fp64 sum of the thread's run of sorted values, then an exclusive scan across the CTA.
      const int base = tid * L;
      double local = 0.0;
#pragma unroll 4
      for (int q = 0; q < L; ++q) {
        int pos = base + q;
        if (pos < n) local = __dadd_rn(local, (double)key_value(keys[pos]));
      }
      double incl = local;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        double o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl = __dadd_rn(incl, o);
      }
      if (lane == 31) warp_sum[warp] = incl;
      __syncthreads();
      double before = 0.0, T = 0.0;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) {
        double ws = warp_sum[w];
        if (w < warp) before = __dadd_rn(before, ws);
        T = __dadd_rn(T, ws);
      }
      double P = __dadd_rn(before, __dsub_rn(incl, local));

      Best best;
      best.D = -1.0;
      best.P = 0.0;
      best.s = 0;
      for (int q = 0; q < L; ++q) {
        int pos = base + q;
        if (pos >= n - 1) break;
        uint32_t kc = keys[pos];
        P = __dadd_rn(P, (double)key_value(kc));
        if (kc == keys[pos + 1]) continue;  // never split a run of equal values
        int s = pos + 1;
        double D = objective(P, T, s, n);
        if (D >= best.D) {  // ascending s: ">=" keeps the largest s among equal objectives
          best.D = D;
          best.P = P;
          best.s = s;
        }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        Best o = shfl_down_best(best, off);
        if (better(o, best)) best = o;
      }
      if (lane == 0) warp_best[warp] = best;
      __syncthreads();
      if (tid == 0) {
        for (int w = 1; w < WARPS; ++w)
          if (better(warp_best[w], best)) best = warp_best[w];
        double m_lo = __ddiv_rn(best.P, (double)best.s);
        double m_hi = __ddiv_rn(__dsub_rn(T, best.P), (double)(n - best.s));
        bool low_side = fabs(m_lo) > fabs(m_hi);  // e marks the partition whose mean is larger in magnitude
        s_tkey = keys[best.s];                    // smallest value of the high partition
        s_mode = low_side ? 1 : 0;
        K_out[row] = low_side ? best.s : n - best.s;
        alpha_out[row] = (float)(low_side ? m_lo : m_hi);
        beta_out[row] = (float)(low_side ? m_hi : m_lo);
        if (flags_out) flags_out[row] = 0u;
      }
    } else if (tid == 0) {
      s_mode = 2;
      s_tkey = 0u;
      K_out[row] = 0;
      float c = bad ? __uint_as_float(0x7FC00000u) : key_value(keys[0]);
      alpha_out[row] = c;
      beta_out[row] = c;
      if (flags_out) flags_out[row] = bad ? DAB_ROW_NONFINITE : DAB_ROW_DEGENERATE;
    }
    __syncthreads();

    const uint32_t tkey = s_tkey;
    const int mode = s_mode;
    for (int w = warp; w < ld_mask; w += WARPS) {
      int i = w * 32 + lane;
      bool bit = false;
      if (mode != 2 && i < n) bit = (order_key(v[i]) >= tkey) != (mode == 1);
      uint32_t word = __ballot_sync(0xFFFFFFFFu, bit);
      if (lane == 0) mrow[w] = word;
    }
    __syncthreads();  // keys and the broadcast slots are reused by the next row
  }
}

template <int NPAD, int THREADS>
static cudaError_t launch_one(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                              float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                              cudaStream_t stream) {
  auto kern = binarize_rows_kernel<NPAD, THREADS>;
  size_t smem = sizeof(uint32_t) * NPAD;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  int64_t grid = rows < (int64_t)(1 << 20) ? rows : (int64_t)(1 << 20);
  kern<<<(unsigned)grid, THREADS, smem, stream>>>(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask, flags);
  return cudaGetLastError();
}

cudaError_t launch_binarize(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                            float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                            cudaStream_t stream) {
#define DAB_CASE(NP, TH) \
  if (n <= NP) return launch_one<NP, TH>(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask, flags, stream)
  DAB_CASE(64, 32);
  DAB_CASE(128, 64);
  DAB_CASE(256, 64);
  DAB_CASE(512, 128);
  DAB_CASE(1024, 128);
  DAB_CASE(2048, 256);
  DAB_CASE(4096, 256);
  DAB_CASE(8192, 512);
  DAB_CASE(16384, 512);
#undef DAB_CASE
  return cudaErrorInvalidValue;
}

}  // namespace dab

// Training-side weight binarization (Algorithm 2, steps 4-13) and the gradient factor of Theorem 4.
//
// Forward: MeanCenter (the mean of a filter's n weights, summed in fp64, is subtracted) and Clamp to [-1, 1]
// give the matrix that is coded; the row coder of binarize.cu codes it; a third kernel writes the dense
// two-level filters W~ = alpha e + beta (1 - e) of Corollary 1.  Backward: per row the l1 norms of the two
// partitions, then the printed expression element by element.  All of it is one pass over 4 n bytes per
// filter: bound by HBM for large layers, by launch latency for the usual few hundred filters.
#include "common.cuh"

namespace dab {
namespace {

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  return v;
}

// One warp per row: Wc = clamp(fp32(w - mean), -1, 1).
__global__ void __launch_bounds__(256) train_center_clamp_kernel(const float* __restrict__ W, int64_t rows, int32_t n,
                                                                 int64_t ld_W, float* __restrict__ Wc, int64_t ld_Wc) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t row = warp0; row < rows; row += nwarps) {
    const float* w = W + row * ld_W;
    double sum = 0.0;
    for (int i = lane; i < n; i += 32) sum += (double)__ldg(w + i);
    const double mean = __ddiv_rn(warp_sum(sum), (double)n);
    float* c = Wc + row * ld_Wc;
    for (int i = lane; i < n; i += 32) {
      const float v = (float)__dsub_rn((double)__ldg(w + i), mean);
      c[i] = fminf(fmaxf(v, -1.0f), 1.0f);
    }
  }
}

// One warp per row: Wt_i = bit i of the row's mask ? alpha : beta.
__global__ void __launch_bounds__(256) train_expand_kernel(const uint32_t* __restrict__ mask, int32_t ld_mask,
                                                           const float* __restrict__ alpha, const float* __restrict__ beta,
                                                           int64_t rows, int32_t n, float* __restrict__ Wt, int64_t ld_Wt) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t row = warp0; row < rows; row += nwarps) {
    const uint32_t* m = mask + row * (int64_t)ld_mask;
    const float a = alpha[row], b = beta[row];
    float* out = Wt + row * ld_Wt;
    for (int i = lane; i < n; i += 32) out[i] = ((__ldg(m + (i >> 5)) >> lane) & 1u) ? a : b;
  }
}

// One warp per row: Theorem 4.  G_i = 1/|part| + (l1 norm of the part / |part|) * STE(W_i), the part being the
// side of the mask element i is on; grad_W_i = grad_Wt_i * G_i.
__global__ void __launch_bounds__(256) train_backward_kernel(const float* __restrict__ Wc, int64_t ld_Wc,
                                                             const uint32_t* __restrict__ mask, int32_t ld_mask,
                                                             const int32_t* __restrict__ K, int64_t rows, int32_t n,
                                                             const float* __restrict__ gWt, int64_t ld_g,
                                                             float* __restrict__ gW, int64_t ld_gw) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t row = warp0; row < rows; row += nwarps) {
    const float* w = Wc + row * ld_Wc;
    const uint32_t* m = mask + row * (int64_t)ld_mask;
    const int k = K[row];
    double l1_sel = 0.0, l1_rest = 0.0;
    for (int i = lane; i < n; i += 32) {
      const double a = fabs((double)__ldg(w + i));
      if ((__ldg(m + (i >> 5)) >> lane) & 1u) l1_sel += a;
      else l1_rest += a;
    }
    l1_sel = warp_sum(l1_sel);
    l1_rest = warp_sum(l1_rest);
    const bool coded = k > 0 && k < n;
    const double inv_sel = coded ? __ddiv_rn(1.0, (double)k) : 0.0, inv_rest = coded ? __ddiv_rn(1.0, (double)(n - k)) : 0.0;
    const double s_sel = coded ? __ddiv_rn(l1_sel, (double)k) : 0.0, s_rest = coded ? __ddiv_rn(l1_rest, (double)(n - k)) : 0.0;
    const float* g = gWt + row * ld_g;
    float* out = gW + row * ld_gw;
    for (int i = lane; i < n; i += 32) {
      const double wi = (double)__ldg(w + i);
      const double ste = fabs(wi) <= 1.0 ? wi : 0.0;
      const bool sel = (__ldg(m + (i >> 5)) >> lane) & 1u;
      const double G = __dadd_rn(sel ? inv_sel : inv_rest, __dmul_rn(sel ? s_sel : s_rest, ste));
      out[i] = (float)__dmul_rn((double)__ldg(g + i), coded ? G : 0.0);
    }
  }
}

unsigned grid_for_rows(int64_t rows) {
  int64_t blocks = (rows + 7) / 8;
  return (unsigned)(blocks > sm_count() * 16 ? sm_count() * 16 : (blocks < 1 ? 1 : blocks));
}

}  // namespace

cudaError_t launch_train_forward(const float* W, int64_t rows, int32_t n, int64_t ld_W, float* Wc, int64_t ld_Wc,
                                 float* Wt, int64_t ld_Wt, int32_t* K, float* alpha, float* beta, uint32_t* mask,
                                 int32_t ld_mask, uint32_t* flags, cudaStream_t stream) {
  train_center_clamp_kernel<<<grid_for_rows(rows), 256, 0, stream>>>(W, rows, n, ld_W, Wc, ld_Wc);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  e = launch_binarize(Wc, rows, n, ld_Wc, K, alpha, beta, mask, ld_mask, flags, stream);
  if (e != cudaSuccess || !Wt) return e;
  train_expand_kernel<<<grid_for_rows(rows), 256, 0, stream>>>(mask, ld_mask, alpha, beta, rows, n, Wt, ld_Wt);
  return cudaGetLastError();
}

cudaError_t launch_train_backward(const float* Wc, int64_t ld_Wc, const uint32_t* mask, int32_t ld_mask,
                                  const int32_t* K, int64_t rows, int32_t n, const float* gWt, int64_t ld_g, float* gW,
                                  int64_t ld_gw, cudaStream_t stream) {
  train_backward_kernel<<<grid_for_rows(rows), 256, 0, stream>>>(Wc, ld_Wc, mask, ld_mask, K, rows, n, gWt, ld_g, gW,
                                                                 ld_gw);
  return cudaGetLastError();
}

}  // namespace dab

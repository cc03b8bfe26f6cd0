// Patch extraction for the general (any geometry) convolution path.
#include "common.cuh"

namespace dab {

// patches[p - patch_begin][c*kh*kw + r*kw + s] = x[img][c][ho*sh - ph + r][wo*sw - pw + s], 0.0 outside.
__global__ void __launch_bounds__(256) im2col_kernel(dab_conv_desc d, int32_t Ho, int32_t Wo,
                                                     const float* __restrict__ x, int64_t patch_begin,
                                                     int64_t patch_count, float* __restrict__ patches) {
  const int32_t n = d.C * d.kh * d.kw;
  const int64_t total = patch_count * n;
  const int32_t khw = d.kh * d.kw;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    int64_t p = patch_begin + idx / n;
    int32_t e = (int32_t)(idx % n);
    int32_t c = e / khw, r = (e % khw) / d.kw, s = e % d.kw;
    int32_t wo = (int32_t)(p % Wo);
    int32_t ho = (int32_t)((p / Wo) % Ho);
    int64_t img = p / ((int64_t)Wo * Ho);
    int32_t h = ho * d.stride_h - d.pad_h + r;
    int32_t w = wo * d.stride_w - d.pad_w + s;
    float v = 0.0f;
    if (h >= 0 && h < d.H && w >= 0 && w < d.W) v = x[((img * d.C + c) * d.H + h) * d.W + w];
    patches[idx] = v;
  }
}

cudaError_t launch_im2col(const dab_conv_desc& d, int32_t Ho, int32_t Wo, const float* x, int64_t patch_begin,
                          int64_t patch_count, float* patches, cudaStream_t stream) {
  int64_t total = patch_count * (int64_t)d.C * d.kh * d.kw;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  if (blocks < 1) blocks = 1;
  im2col_kernel<<<(unsigned)blocks, 256, 0, stream>>>(d, Ho, Wo, x, patch_begin, patch_count, patches);
  return cudaGetLastError();
}

}  // namespace dab

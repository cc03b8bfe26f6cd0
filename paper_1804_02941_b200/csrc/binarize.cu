// dab_binarize (rows of a matrix) and the patch coder of dab_binary_conv (patches of an NCHW tensor).
// Both drive the same group-of-warps row coder (rowcode.cuh); they differ in where a row's values come from
// and where the results go.
#include "rowcode.cuh"

namespace dab {

// Writes the packed mask of one row: the group's warps take 32-word batches; lane t keeps word t of a batch so
// that a batch is stored with one coalesced write.  Words between ceil(n/32) and ld are written as 0.
template <int W, typename Value>
__device__ __forceinline__ void group_write_mask(Value value, int n, int ld, const RowResult& res, int tig,
                                                 uint32_t* __restrict__ out) {
  const int lane = tig & 31, warp = tig >> 5;
  const bool flip = res.mode == 1;
  for (int w0 = warp * 32; w0 < ld; w0 += 32 * W) {
    uint32_t mine = 0;
    const int wend = min(32, ld - w0);
    for (int t = 0; t < wend; ++t) {
      int i = (w0 + t) * 32 + lane;
      bool bit = false;
      if (res.mode != 2 && i < n) bit = (order_key(value(i)) >= res.tkey) != flip;
      uint32_t word = __ballot_sync(0xFFFFFFFFu, bit);
      if (lane == t) mine = word;
    }
    if (lane < wend) out[w0 + lane] = mine;
  }
}

__host__ __device__ inline int scratch_words_for(int n, int W) {
  int cap = 128 * W;
  while (cap < n) cap <<= 1;
  return cap + (cap >> 5) + 1;
}

// ---------------------------------------------------------------------------------------------------------
// Rows of a matrix.  A CTA of WARPS warps holds WARPS/W groups; each group walks over rows.
// ---------------------------------------------------------------------------------------------------------
template <int W, int WARPS>
__global__ void __launch_bounds__(WARPS * 32) binarize_rows_kernel(const float* __restrict__ values, int64_t rows,
                                                                   int32_t n, int64_t ld_values,
                                                                   int32_t* __restrict__ K_out,
                                                                   float* __restrict__ alpha_out,
                                                                   float* __restrict__ beta_out,
                                                                   uint32_t* __restrict__ mask_out, int32_t ld_mask,
                                                                   uint32_t* __restrict__ flags_out,
                                                                   int scratch_words) {
  constexpr int G = WARPS / W;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  GroupShared* gs_all = reinterpret_cast<GroupShared*>(smem_raw);
  uint32_t* scratch_all = reinterpret_cast<uint32_t*>(smem_raw + sizeof(GroupShared) * G);

  const int group = threadIdx.x / (32 * W);
  const int tig = threadIdx.x % (32 * W);
  GroupShared* gs = gs_all + group;
  uint32_t* scratch = scratch_all + (size_t)group * scratch_words;
  const int bar_id = 1 + group;

  for (int64_t row = (int64_t)blockIdx.x * G + group; row < rows; row += (int64_t)gridDim.x * G) {
    const float* v = values + row * ld_values;
    auto value = [v](int i) { return __ldg(v + i); };
    group_code_row<W>(value, n, tig, scratch, gs, bar_id);
    const RowResult res = gs->result;
    if (tig == 0) {
      K_out[row] = res.K;
      alpha_out[row] = res.alpha;
      beta_out[row] = res.beta;
      if (flags_out) flags_out[row] = res.flags;
    }
    group_write_mask<W>(value, n, ld_mask, res, tig, mask_out + row * (int64_t)ld_mask);
    group_barrier(bar_id, 32 * W);  // gs->result is overwritten by the next row
  }
}

template <int W, int WARPS>
static cudaError_t launch_rows(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                               float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                               cudaStream_t stream) {
  constexpr int G = WARPS / W;
  auto kern = binarize_rows_kernel<W, WARPS>;
  int sw = scratch_words_for(n, W);
  size_t smem = sizeof(GroupShared) * G + sizeof(uint32_t) * (size_t)sw * G;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int64_t blocks = (rows + G - 1) / G;
  const int64_t cap = 148 * 16;
  if (blocks > cap) blocks = cap;
  kern<<<(unsigned)blocks, WARPS * 32, smem, stream>>>(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask,
                                                       flags, sw);
  return cudaGetLastError();
}

cudaError_t launch_binarize(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K,
                            float* alpha, float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags,
                            cudaStream_t stream) {
#define DAB_ROWS(Wv, WARPSv) \
  return launch_rows<Wv, WARPSv>(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask, flags, stream)
  if (n <= 1024) DAB_ROWS(1, 8);
  if (n <= 2048) DAB_ROWS(2, 8);
  if (n <= 4096) DAB_ROWS(4, 8);
  if (n <= 8192) DAB_ROWS(8, 8);
  DAB_ROWS(16, 16);
#undef DAB_ROWS
}

// ---------------------------------------------------------------------------------------------------------
// Patches of an NCHW tensor.  A CTA stages the input region under a tile of TH x TW output positions (all
// channels, zero padding filled in) in shared memory, then its groups code the tile's patches one by one.
// Element i of a patch, i = (c*kh + r)*kw + s, sits at tile offset off[i] + patch origin.
// ---------------------------------------------------------------------------------------------------------
struct PatchArgs {
  dab_conv_desc d;
  int32_t Ho, Wo, n;
  int32_t TH, TW;          // output positions per tile
  int32_t in_h, in_w;      // staged rows/columns per channel: (TH-1)*stride_h + kh, (TW-1)*stride_w + kw
  int32_t pitch;           // words per staged row (>= in_w)
  int32_t tiles_h, tiles_w;
  int32_t scratch_words;
  const float* x;
  int32_t* pK;
  float* pgamma;
  float* pdelta;
  uint32_t* pflags;        // may be null
  uint32_t* pmask;
  int32_t ldp;
};

template <int W, int WARPS>
__global__ void __launch_bounds__(WARPS * 32) binarize_patches_kernel(const PatchArgs a) {
  constexpr int G = WARPS / W;
  constexpr int THREADS = WARPS * 32;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  GroupShared* gs_all = reinterpret_cast<GroupShared*>(smem_raw);
  uint32_t* scratch_all = reinterpret_cast<uint32_t*>(smem_raw + sizeof(GroupShared) * G);
  float* tile = reinterpret_cast<float*>(scratch_all + (size_t)G * a.scratch_words);
  const int ch_words = a.in_h * a.pitch;
  uint16_t* off = reinterpret_cast<uint16_t*>(tile + (size_t)a.d.C * ch_words);

  const int group = threadIdx.x / (32 * W);
  const int tig = threadIdx.x % (32 * W);
  GroupShared* gs = gs_all + group;
  uint32_t* scratch = scratch_all + (size_t)group * a.scratch_words;
  const int bar_id = 1 + group;

  // element offsets inside the tile (same for every patch)
  const int khw = a.d.kh * a.d.kw;
  for (int i = threadIdx.x; i < a.n; i += THREADS) {
    int c = i / khw, rs = i % khw;
    off[i] = (uint16_t)(c * ch_words + (rs / a.d.kw) * a.pitch + (rs % a.d.kw));
  }

  const int64_t tiles_per_img = (int64_t)a.tiles_h * a.tiles_w;
  const int64_t total_tiles = tiles_per_img * a.d.N;
  for (int64_t tile_id = blockIdx.x; tile_id < total_tiles; tile_id += gridDim.x) {
    const int img = (int)(tile_id / tiles_per_img);
    const int trem = (int)(tile_id % tiles_per_img);
    const int ho0 = (trem / a.tiles_w) * a.TH, wo0 = (trem % a.tiles_w) * a.TW;
    const int h0 = ho0 * a.d.stride_h - a.d.pad_h, w0 = wo0 * a.d.stride_w - a.d.pad_w;

    __syncthreads();  // the previous tile is no longer read
    const float* ximg = a.x + (int64_t)img * a.d.C * a.d.H * a.d.W;
    const int per_ch = a.in_h * a.in_w;
    for (int idx = threadIdx.x; idx < a.d.C * per_ch; idx += THREADS) {
      int c = idx / per_ch, rem = idx % per_ch;
      int r = rem / a.in_w, s = rem % a.in_w;
      int h = h0 + r, w = w0 + s;
      float v = 0.0f;
      if (h >= 0 && h < a.d.H && w >= 0 && w < a.d.W) v = __ldg(ximg + ((int64_t)c * a.d.H + h) * a.d.W + w);
      tile[c * ch_words + r * a.pitch + s] = v;
    }
    __syncthreads();

    const int th = min(a.TH, a.Ho - ho0), tw = min(a.TW, a.Wo - wo0);
    for (int p = group; p < th * tw; p += G) {
      const int lh = p / tw, lw = p % tw;
      const float* origin = tile + lh * a.d.stride_h * a.pitch + lw * a.d.stride_w;
      auto value = [origin, off](int i) { return origin[off[i]]; };
      group_code_row<W>(value, a.n, tig, scratch, gs, bar_id);
      const RowResult res = gs->result;
      const int64_t pi = ((int64_t)img * a.Ho + (ho0 + lh)) * a.Wo + (wo0 + lw);
      if (tig == 0) {
        a.pK[pi] = res.K;
        a.pgamma[pi] = res.alpha;
        a.pdelta[pi] = res.beta;
        if (a.pflags) a.pflags[pi] = res.flags;
      }
      group_write_mask<W>(value, a.n, a.ldp, res, tig, a.pmask + pi * (int64_t)a.ldp);
      group_barrier(bar_id, 32 * W);
    }
  }
}

// Picks the tile: the largest of a few shapes whose staged input fits the shared-memory budget.
static void choose_tile(const dab_conv_desc& d, int Ho, int Wo, size_t budget_bytes, PatchArgs* a) {
  static const int shapes[][2] = {{8, 8}, {4, 8}, {4, 4}, {2, 4}, {2, 2}, {1, 2}, {1, 1}};
  for (auto& sh : shapes) {
    int TH = sh[0] < Ho ? sh[0] : Ho, TW = sh[1] < Wo ? sh[1] : Wo;
    int in_h = (TH - 1) * d.stride_h + d.kh, in_w = (TW - 1) * d.stride_w + d.kw;
    int pitch = in_w | 1;  // odd pitch spreads the rows of a patch over the banks
    size_t bytes = (size_t)d.C * in_h * pitch * sizeof(float);
    if (bytes <= budget_bytes || (TH == 1 && TW == 1)) {
      a->TH = TH; a->TW = TW; a->in_h = in_h; a->in_w = in_w; a->pitch = pitch;
      a->tiles_h = (Ho + TH - 1) / TH; a->tiles_w = (Wo + TW - 1) / TW;
      return;
    }
  }
}

template <int W, int WARPS>
static cudaError_t launch_patches_t(PatchArgs& a, cudaStream_t stream) {
  constexpr int G = WARPS / W;
  auto kern = binarize_patches_kernel<W, WARPS>;
  a.scratch_words = scratch_words_for(a.n, W);
  size_t fixed = sizeof(GroupShared) * G + sizeof(uint32_t) * (size_t)a.scratch_words * G + sizeof(uint16_t) * a.n + 16;
  const size_t limit = 200 * 1024;
  size_t budget = limit > fixed ? limit - fixed : 0;
  if (budget > 72 * 1024) budget = 72 * 1024;  // leave room for more than one CTA per SM when the tile is small
  choose_tile(a.d, a.Ho, a.Wo, budget, &a);
  size_t tile_bytes = (size_t)a.d.C * a.in_h * a.pitch * sizeof(float);
  if ((size_t)a.d.C * a.in_h * a.pitch > 65535) return cudaErrorInvalidValue;  // offsets are 16-bit
  size_t smem = fixed + tile_bytes;
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int64_t tiles = (int64_t)a.tiles_h * a.tiles_w * a.d.N;
  int64_t blocks = tiles < 148 * 8 ? tiles : 148 * 8;
  kern<<<(unsigned)blocks, WARPS * 32, smem, stream>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_binarize_patches(const dab_conv_desc& d, int32_t Ho, int32_t Wo, const float* x, int32_t* pK,
                                    float* pgamma, float* pdelta, uint32_t* pmask, int32_t ldp, uint32_t* pflags,
                                    cudaStream_t stream) {
  PatchArgs a;
  a.d = d; a.Ho = Ho; a.Wo = Wo; a.n = d.C * d.kh * d.kw;
  a.x = x; a.pK = pK; a.pgamma = pgamma; a.pdelta = pdelta; a.pflags = pflags; a.pmask = pmask; a.ldp = ldp;
  if (a.n <= 1024) return launch_patches_t<1, 8>(a, stream);
  if (a.n <= 2048) return launch_patches_t<2, 8>(a, stream);
  if (a.n <= 4096) return launch_patches_t<4, 8>(a, stream);
  if (a.n <= 8192) return launch_patches_t<8, 8>(a, stream);
  return launch_patches_t<16, 16>(a, stream);
}

}  // namespace dab

// The patch coder of dab_binary_conv: the row coder of rowcode.cuh applied to every patch of an NCHW tensor
// (one warp per patch for up to 1024 values, a group of 2..16 warps beyond).
#include <atomic>

#include "histcode.cuh"
#include "rowcode.cuh"

namespace dab {

// ---------------------------------------------------------------------------------------------------------
// Patches of an NCHW tensor.  A CTA stages the input region under a tile of TH x TW output positions (all
// channels, zero padding filled in) in shared memory, then codes the tile's patches.
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
  int32_t defer_dense;     // leave tiles that look dense to the next kernel of the chain (marks them in pK)
  int32_t dense_num, dense_den;  // a tile is dense if non-zero staged values * dense_den > staged values * dense_num
  int32_t marked_only;     // code only the tiles marked by the kernel before (chains of kernels on one stream hand
                           // tiles on through marks; a CTA none of whose tiles is marked leaves at entry)
  int32_t tile_shape;      // index into kTileShapes forced by the caller, -1: choose
  uint32_t magic_per_ch, magic_in_w;  // ceil(2^32 / d) for d = in_h*in_w and in_w: floor(i/d) = umulhi(i, magic); 0 if d == 1
  const float* x;
  int32_t* pK;
  float* pgamma;
  float* pdelta;
  uint32_t* pflags;        // may be null
  uint32_t* pmask;
  int32_t ldp;
};

// Extents of the arrays of a call (what the checked indices of a debug build are compared with).
__device__ __forceinline__ int64_t patch_count(const PatchArgs& a) { return (int64_t)a.d.N * a.Ho * a.Wo; }
__device__ __forceinline__ int64_t image_values(const PatchArgs& a) { return (int64_t)a.d.C * a.d.H * a.d.W; }

__device__ __forceinline__ void fill_offsets(const PatchArgs& a, uint16_t* off, int ch_words, int tid, int threads) {
  const int khw = a.d.kh * a.d.kw;
  for (int i = tid; i < a.n; i += threads) {
    int c = i / khw, rs = i % khw;
    off[i] = (uint16_t)(c * ch_words + (rs / a.d.kw) * a.pitch + (rs % a.d.kw));
  }
}

// Stages the tile whose first input row/column is (h0, w0) of image `ximg`; out-of-image positions become 0.0.
// Returns the number of non-zero values this thread staged.  kKeys: the tile holds the order-preserving keys of the
// values (each element is part of up to kh*kw patches: its key is computed once here, not once per patch).
template <bool kKeys>
__device__ __forceinline__ int load_tile(const PatchArgs& a, const float* __restrict__ ximg, int h0, int w0,
                                         float* tile, int ch_words, int tid, int threads) {
  const int per_ch = a.in_h * a.in_w;
  const int total = a.d.C * per_ch;
  int nonzero = 0;
  for (int idx = tid; idx < total; idx += threads) {
    int c = a.magic_per_ch ? (int)__umulhi((unsigned)idx, a.magic_per_ch) : idx;  // magic 0: divisor 1
    int rem = idx - c * per_ch;
    int r = a.magic_in_w ? (int)__umulhi((unsigned)rem, a.magic_in_w) : rem;
    int s = rem - r * a.in_w;
    int h = h0 + r, w = w0 + s;
    float v = 0.0f;
    if ((unsigned)h < (unsigned)a.d.H && (unsigned)w < (unsigned)a.d.W)
      v = __ldg(ximg + DAB_IDX(((int64_t)c * a.d.H + h) * a.d.W + w, image_values(a)));
    tile[c * ch_words + r * a.pitch + s] = kKeys ? __uint_as_float(order_key(v)) : v;
    nonzero += (v != 0.0f);
  }
  return nonzero;
}

// Index of the first patch of a tile: where the one-warp kernel leaves its "dense tile" mark (K = -1, a value no
// coded patch has) for the group kernel that follows it on the stream.
constexpr int32_t kDenseMark = -1;

struct TileCoord {
  int img, ho0, wo0, h0, w0, th, tw;
};

__device__ __forceinline__ TileCoord tile_coord(const PatchArgs& a, int64_t tile_id) {
  const int64_t tiles_per_img = (int64_t)a.tiles_h * a.tiles_w;
  TileCoord t;
  t.img = (int)(tile_id / tiles_per_img);
  const int trem = (int)(tile_id % tiles_per_img);
  t.ho0 = (trem / a.tiles_w) * a.TH;
  t.wo0 = (trem % a.tiles_w) * a.TW;
  t.h0 = t.ho0 * a.d.stride_h - a.d.pad_h;
  t.w0 = t.wo0 * a.d.stride_w - a.d.pad_w;
  t.th = min(a.TH, a.Ho - t.ho0);
  t.tw = min(a.TW, a.Wo - t.wo0);
  return t;
}

// Staged values of a tile that come from the image (the rest is zero padding): what its density is measured on.
__device__ __forceinline__ int64_t staged_inside(const PatchArgs& a, const TileCoord& t) {
  const int rows = min(t.h0 + a.in_h, a.d.H) - max(t.h0, 0), cols = min(t.w0 + a.in_w, a.d.W) - max(t.w0, 0);
  return (int64_t)a.d.C * max(rows, 0) * max(cols, 0);
}

// Whether a marked-only kernel has anything to do in this CTA: the marks of the CTA's own tiles are read, one tile
// per thread at a time.  Every thread of the CTA gets the same answer.
__device__ __forceinline__ bool has_marked_tile(const PatchArgs& a) {
  const int64_t total_tiles = (int64_t)a.tiles_h * a.tiles_w * a.d.N;
  int any = 0;
  for (int64_t tile_id = blockIdx.x + (int64_t)threadIdx.x * gridDim.x; tile_id < total_tiles;
       tile_id += (int64_t)blockDim.x * gridDim.x) {
    const TileCoord t = tile_coord(a, tile_id);
    any |= a.pK[DAB_IDX(((int64_t)t.img * a.Ho + t.ho0) * a.Wo + t.wo0, patch_count(a))] == kDenseMark;
  }
  return __syncthreads_or(any) != 0;
}

#ifndef DAB_WARP_MINBLOCKS
#define DAB_WARP_MINBLOCKS 3  // CTAs per SM the one-warp-per-patch kernel is compiled for (register budget)
#endif

template <int R, bool kFull>
__global__ void __launch_bounds__(kWarpsPerCta * 32, DAB_WARP_MINBLOCKS) binarize_patches_warp_kernel(const PatchArgs a) {
  constexpr int THREADS = kWarpsPerCta * 32;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* rcp = reinterpret_cast<double*>(smem_raw);
  uint32_t* scratch_all = reinterpret_cast<uint32_t*>(rcp + rcp_table_slots(a.n));
  float* tile = reinterpret_cast<float*>(scratch_all + kWarpsPerCta * 32 * R);
  const int ch_words = a.in_h * a.pitch;
  uint16_t* off = reinterpret_cast<uint16_t*>(tile + (size_t)a.d.C * ch_words);

  __shared__ int tile_nonzero;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* scratch = scratch_all + warp * (32 * R);
  fill_reciprocals(rcp, a.n, threadIdx.x, THREADS);
  fill_offsets(a, off, ch_words, threadIdx.x, THREADS);

  const int64_t total_tiles = (int64_t)a.tiles_h * a.tiles_w * a.d.N;
  for (int64_t tile_id = blockIdx.x; tile_id < total_tiles; tile_id += gridDim.x) {
    const TileCoord t = tile_coord(a, tile_id);
    __syncthreads();  // the previous tile is no longer read
    if (threadIdx.x == 0) tile_nonzero = 0;
    int nz = load_tile<true>(a, a.x + (int64_t)t.img * a.d.C * a.d.H * a.d.W, t.h0, t.w0, tile, ch_words, threadIdx.x,
                       THREADS);
    const int64_t first_patch = ((int64_t)t.img * a.Ho + t.ho0) * a.Wo + t.wo0;
    if (a.defer_dense) {
      // One warp per patch suits patches whose non-zero values fit 8 keys per lane (at most 256).  A tile whose
      // density says otherwise (expected non-zeros per patch = density of the staged region * n > 256) is left to
      // the group kernel, which sorts it with about 8 keys per thread again.
      __syncthreads();
      nz = __reduce_add_sync(0xFFFFFFFFu, nz);
      if (lane == 0 && nz) atomicAdd(&tile_nonzero, nz);
      __syncthreads();
      const int64_t staged = staged_inside(a, t);
      if ((int64_t)tile_nonzero * a.dense_den > a.dense_num * staged) {
        if (threadIdx.x == 0 && DAB_IN_BOUNDS(first_patch, patch_count(a))) a.pK[first_patch] = kDenseMark;
        continue;
      }
    } else {
      __syncthreads();
    }

    for (int p = warp; p < t.th * t.tw; p += kWarpsPerCta) {
      const int lh = p / t.tw, lw = p % t.tw;
      const float* origin = tile + lh * a.d.stride_h * a.pitch + lw * a.d.stride_w;
      auto keyof = [origin, off](int i) { return __float_as_uint(origin[off[i]]); };
      uint32_t kreg[R];
      RowResult res = warp_code_row<R, kFull>(keyof, a.n, lane, scratch, rcp, kreg);
      const int64_t pi = ((int64_t)t.img * a.Ho + (t.ho0 + lh)) * a.Wo + (t.wo0 + lw);
      if (lane == 0 && DAB_IN_BOUNDS(pi, patch_count(a))) {
        a.pK[pi] = res.K;
        a.pgamma[pi] = res.alpha;
        a.pdelta[pi] = res.beta;
        if (a.pflags) a.pflags[pi] = res.flags;
      }
      uint32_t mine = warp_mask_words<R, kFull>(kreg, a.n, lane, res);
      uint32_t* mrow = a.pmask + pi * (int64_t)a.ldp;
      for (int w = lane; w < a.ldp; w += 32)
        if (DAB_IN_BOUNDS(pi * a.ldp + w, patch_count(a) * a.ldp)) mrow[w] = (w < 32) ? mine : 0u;
    }
  }
}

template <int W, int WARPS, int R, bool kFull, bool kTable>
__global__ void __launch_bounds__(WARPS * 32) binarize_patches_group_kernel(const PatchArgs a) {
  constexpr int G = WARPS / W;
  constexpr int THREADS = WARPS * 32;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* rcp = reinterpret_cast<double*>(smem_raw);
  GroupShared* gs_all = reinterpret_cast<GroupShared*>(rcp + (kTable ? rcp_table_slots(a.n) : 0));
  uint32_t* scratch_all = reinterpret_cast<uint32_t*>(gs_all + G);
  float* tile = reinterpret_cast<float*>(scratch_all + (size_t)G * a.scratch_words);
  const int ch_words = a.in_h * a.pitch;
  uint16_t* off = reinterpret_cast<uint16_t*>(tile + (size_t)a.d.C * ch_words);

  const int group = threadIdx.x / (32 * W);
  const int tig = threadIdx.x % (32 * W);
  GroupShared* gs = gs_all + group;
  uint32_t* scratch = scratch_all + (size_t)group * a.scratch_words;
  const int bar_id = 1 + group;
  if (a.marked_only && !has_marked_tile(a)) return;
  __shared__ int tile_nonzero;
  if (kTable) fill_reciprocals(rcp, a.n, threadIdx.x, THREADS);
  fill_offsets(a, off, ch_words, threadIdx.x, THREADS);

  const int64_t total_tiles = (int64_t)a.tiles_h * a.tiles_w * a.d.N;
  for (int64_t tile_id = blockIdx.x; tile_id < total_tiles; tile_id += gridDim.x) {
    const TileCoord t = tile_coord(a, tile_id);
    const int64_t first_patch = ((int64_t)t.img * a.Ho + t.ho0) * a.Wo + t.wo0;
    if (a.marked_only && a.pK[DAB_IDX(first_patch, patch_count(a))] != kDenseMark) continue;
    __syncthreads();
    if (threadIdx.x == 0) tile_nonzero = 0;
    int nz = load_tile<true>(a, a.x + (int64_t)t.img * a.d.C * a.d.H * a.d.W, t.h0, t.w0, tile, ch_words, threadIdx.x,
                             THREADS);
    __syncthreads();
    if (a.defer_dense) {  // dense tiles go to the next kernel of the chain
      nz = __reduce_add_sync(0xFFFFFFFFu, nz);
      if ((threadIdx.x & 31) == 0 && nz) atomicAdd(&tile_nonzero, nz);
      __syncthreads();
      const int64_t staged = staged_inside(a, t);
      if ((int64_t)tile_nonzero * a.dense_den > a.dense_num * staged) {
        if (threadIdx.x == 0 && DAB_IN_BOUNDS(first_patch, patch_count(a))) a.pK[first_patch] = kDenseMark;
        continue;
      }
    }

    for (int p = group; p < t.th * t.tw; p += G) {
      const int lh = p / t.tw, lw = p % t.tw;
      const float* origin = tile + lh * a.d.stride_h * a.pitch + lw * a.d.stride_w;
      auto keyof = [origin, off](int i) { return __float_as_uint(origin[off[i]]); };
      uint32_t kreg[R];
      group_code_row<W, R, kFull, kTable>(keyof, a.n, tig, scratch, gs, bar_id, rcp, kreg);
      const RowResult res = gs->result;
      const int64_t pi = ((int64_t)t.img * a.Ho + (t.ho0 + lh)) * a.Wo + (t.wo0 + lw);
      if (tig == 0 && DAB_IN_BOUNDS(pi, patch_count(a))) {
        a.pK[pi] = res.K;
        a.pgamma[pi] = res.alpha;
        a.pdelta[pi] = res.beta;
        if (a.pflags) a.pflags[pi] = res.flags;
      }
      group_store_mask<W, R, kFull>(kreg, a.n, a.ldp, tig, res, a.pmask, pi, patch_count(a));
      group_barrier(bar_id, 32 * W);
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// Histogram-pruned patch coder: the search of histcode.cuh, one warp per patch, on the staged tile (one
// quantisation per tile, from the range of its non-zero values), then the mask as a threshold compare as in
// the other coders.  Patches the search does not settle, and tiles holding a NaN or an infinity, are left to the
// group kernel through the dense-tile mark.
// ---------------------------------------------------------------------------------------------------------
struct HistTile {          // per tile, in shared memory
  uint32_t kmin, kmax;     // smallest and largest key among the non-zero staged values
  int retry;               // some patch of the tile could not be coded here
};

#ifndef DAB_HIST_MINBLOCKS
#define DAB_HIST_MINBLOCKS 3  // CTAs per SM the histogram coder is compiled for (register budget)
#endif

// KHW: kh*kw when it is 9 (the sweeps over a patch are then fully unrolled over the kernel window), 0 otherwise.
template <int BPL, int KHW>
__global__ void __launch_bounds__(kWarpsPerCta * 32, DAB_HIST_MINBLOCKS) binarize_patches_hist_kernel(const PatchArgs a) {
  constexpr int THREADS = kWarpsPerCta * 32;
  constexpr int B = 32 * BPL;
  constexpr int LOG2B = BPL == 1 ? 5 : BPL == 2 ? 6 : BPL == 4 ? 7 : 8;
  constexpr int KMAX = KHW ? KHW : 1;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* rcp = reinterpret_cast<double*>(smem_raw);
  int2* hist_all = reinterpret_cast<int2*>(rcp + rcp_table_slots(a.n));          // [warp][B] (count, sum of offsets)
  uint32_t* scratch_all = reinterpret_cast<uint32_t*>(hist_all + kWarpsPerCta * B);
  float* tile = reinterpret_cast<float*>(scratch_all + kWarpsPerCta * hist_cap(BPL));
  const int ch_words = (a.in_h * a.pitch) | 1;  // odd: the 32 channels a warp reads at once fall into 32 banks
  uint16_t* off = reinterpret_cast<uint16_t*>(tile + (size_t)a.d.C * ch_words);
  uint16_t* win = off + ((a.n + 1) & ~1);       // offsets of the kernel window inside one channel
  __shared__ HistTile ht;

  if (a.marked_only && !has_marked_tile(a)) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int2* hist = hist_all + warp * B;
  uint32_t* scratch = scratch_all + warp * hist_cap(BPL);
  const int khw = a.d.kh * a.d.kw;
  fill_reciprocals(rcp, a.n, threadIdx.x, THREADS);
  fill_offsets(a, off, ch_words, threadIdx.x, THREADS);
  for (int rs = threadIdx.x; rs < khw; rs += THREADS) win[rs] = (uint16_t)((rs / a.d.kw) * a.pitch + rs % a.d.kw);
  __syncthreads();
  int wofs[KMAX];
#pragma unroll
  for (int rs = 0; rs < KMAX; ++rs) wofs[rs] = KHW ? win[rs] : 0;
  const int qbits = quant_bits(a.n, LOG2B);
  const int rounds = (a.n + 31) >> 5;

  const int64_t total_tiles = (int64_t)a.tiles_h * a.tiles_w * a.d.N;
  for (int64_t tile_id = blockIdx.x; tile_id < total_tiles; tile_id += gridDim.x) {
    const TileCoord t = tile_coord(a, tile_id);
    if (a.marked_only && a.pK[DAB_IDX(((int64_t)t.img * a.Ho + t.ho0) * a.Wo + t.wo0, patch_count(a))] != kDenseMark) continue;
    __syncthreads();  // the previous tile is no longer read
    if (threadIdx.x == 0) { ht.kmin = kPadKey; ht.kmax = 0u; ht.retry = 0; }
    __syncthreads();
    {  // stage the values (-0.0 folded onto +0.0) and find the range of the non-zero ones
      const float* ximg = a.x + (int64_t)t.img * a.d.C * a.d.H * a.d.W;
      const int per_ch = a.in_h * a.in_w, total = a.d.C * per_ch;
      uint32_t kmin = kPadKey, kmax = 0u;
      for (int idx = threadIdx.x; idx < total; idx += THREADS) {
        int c = a.magic_per_ch ? (int)__umulhi((unsigned)idx, a.magic_per_ch) : idx;
        int rem = idx - c * per_ch;
        int r = a.magic_in_w ? (int)__umulhi((unsigned)rem, a.magic_in_w) : rem;
        int s = rem - r * a.in_w;
        int h = t.h0 + r, w = t.w0 + s;
        float v = 0.0f;
        if ((unsigned)h < (unsigned)a.d.H && (unsigned)w < (unsigned)a.d.W)
          v = __fadd_rn(__ldg(ximg + DAB_IDX(((int64_t)c * a.d.H + h) * a.d.W + w, image_values(a))), 0.0f);
        tile[c * ch_words + r * a.pitch + s] = v;
        if (v != 0.0f) {  // NaN compares unequal: counted, and seen as non-finite below
          const uint32_t key = order_key(v);
          kmin = min(kmin, key);
          kmax = max(kmax, key);
        }
      }
      kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
      kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
      if (lane == 0 && kmin <= kmax) {
        atomicMin(&ht.kmin, kmin);
        atomicMax(&ht.kmax, kmax);
      }
    }
    __syncthreads();
    const int64_t first_patch = ((int64_t)t.img * a.Ho + t.ho0) * a.Wo + t.wo0;
    const uint32_t tkmin = ht.kmin, tkmax = ht.kmax;
    const bool any_nonzero = tkmin <= tkmax;
    if (any_nonzero && key_range_nonfinite(tkmin, tkmax)) {
      if (threadIdx.x == 0 && DAB_IN_BOUNDS(first_patch, patch_count(a))) a.pK[first_patch] = kDenseMark;
      continue;
    }
    const float lo = any_nonzero ? key_value(tkmin) : 0.0f, hi = any_nonzero ? key_value(tkmax) : 0.0f;
    const Quant qz = make_quant(lo, hi, qbits, LOG2B);  // one quantisation for the tile

    for (int p = warp; p < t.th * t.tw; p += kWarpsPerCta) {
      const int lh = p / t.tw, lw = p % t.tw;
      const float* origin = tile + lh * a.d.stride_h * a.pitch + lw * a.d.stride_w;
      const int64_t pi = ((int64_t)t.img * a.Ho + (t.ho0 + lh)) * a.Wo + (t.wo0 + lw);
      uint32_t* mrow = a.pmask + pi * (int64_t)a.ldp;

      // the two sweeps of the search take the elements in any order: lane = channel, loop over the kernel window
      auto sweep = [&](auto f) {
        for (int c0 = 0; c0 < a.d.C; c0 += 32) {
          const bool cin = c0 + lane < a.d.C;
          const float* src = origin + (cin ? c0 + lane : 0) * ch_words;
          if (KHW) {
#pragma unroll
            for (int rs = 0; rs < KMAX; ++rs) f(src[wofs[rs]], cin);
          } else {
            for (int rs = 0; rs < khw; ++rs) f(src[win[rs]], cin);
          }
        }
      };
      RowResult res;
      const bool retry = !hist_search<BPL>(sweep, a.n, qz, hist, scratch, rcp, lane, res);
      if (retry) {
        if (lane == 0) ht.retry = 1;
        continue;
      }
      // ---- pass 3: outputs (mask bits in element order, through the offset table) ----
      if (lane == 0 && DAB_IN_BOUNDS(pi, patch_count(a))) {
        a.pK[pi] = res.K;
        a.pgamma[pi] = res.alpha;
        a.pdelta[pi] = res.beta;
        if (a.pflags) a.pflags[pi] = res.flags;
      }
      const bool flip = res.mode == 1, none = res.mode == 2;
      const float tv = key_value(res.tkey);
      const bool keep = !none;
      for (int kb = 0; kb < rounds; kb += 32) {  // 32 mask words at a time: word kb + j ends up in lane j
        const int kend = min(32, rounds - kb);
        uint32_t mine = 0;
#pragma unroll 6
        for (int kk = 0; kk < kend; ++kk) {
          const int i = (kb + kk) * 32 + lane;
          const bool live = i < a.n;
          const float v = origin[live ? off[i] : 0];
          const uint32_t word = __ballot_sync(0xFFFFFFFFu, keep && live && ((v >= tv) != flip));
          if (kk == lane) mine = word;
        }
        if (lane < kend && DAB_IN_BOUNDS(pi * a.ldp + kb + lane, patch_count(a) * a.ldp)) mrow[kb + lane] = mine;
      }
      for (int w = rounds + lane; w < a.ldp; w += 32)
        if (DAB_IN_BOUNDS(pi * a.ldp + w, patch_count(a) * a.ldp)) mrow[w] = 0u;
    }
    __syncthreads();
    if (threadIdx.x == 0 && ht.retry && DAB_IN_BOUNDS(first_patch, patch_count(a))) a.pK[first_patch] = kDenseMark;
  }
}

// ---------------------------------------------------------------------------------------------------------
// Sign coding (the paper's XNOR-structured FBin inputs): mask bit = [x >= 0], gamma = mean |x|, delta = -gamma.
// One warp per row; `value(i)` returns element i.  HBM-bound work: no sort, one pass.
// ---------------------------------------------------------------------------------------------------------
template <typename Value>
__device__ __forceinline__ void warp_sign_row(Value value, int n, int ld, int lane, int32_t* K_out, float* gamma_out,
                                              float* delta_out, uint32_t* flags_out, uint32_t* __restrict__ mrow) {
  double sum = 0.0;
  int ones = 0, bad = 0;
  uint32_t mine = 0;
  const int words = (n + 31) >> 5;
  for (int k = 0; k < words; ++k) {
    const int i = k * 32 + lane;
    float x = -1.0f;  // lanes beyond n contribute a 0 bit
    if (i < n) {
      x = value(i);
      bad |= is_nonfinite(x);
      sum += fabs((double)x);
    }
    const uint32_t word = __ballot_sync(0xFFFFFFFFu, i < n && x >= 0.0f);
    ones += __popc(word);
    if ((k & 31) == lane) mine = word;
    if ((k & 31) == 31 || k == words - 1) {  // a batch of up to 32 words is complete: one coalesced store
      const int w = (k & ~31) + lane;
      if (w <= k) mrow[w] = mine;
    }
  }
  for (int w = words + lane; w < ld; w += 32) mrow[w] = 0u;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, off);
  bad = __any_sync(0xFFFFFFFFu, bad);
  if (bad) {  // flagged rows: empty mask, NaN scales
    __syncwarp();
    for (int w = lane; w < ld; w += 32) mrow[w] = 0u;
  }
  if (lane == 0) {
    const float g = bad ? __uint_as_float(0x7FC00000u) : (float)(sum / (double)n);
    *K_out = bad ? 0 : ones;
    *gamma_out = g;
    *delta_out = -g;
    if (flags_out) *flags_out = bad ? DAB_ROW_NONFINITE : 0u;
  }
}

__global__ void __launch_bounds__(kWarpsPerCta * 32) sign_patches_kernel(const PatchArgs a) {
  constexpr int THREADS = kWarpsPerCta * 32;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* tile = reinterpret_cast<float*>(smem_raw);
  const int ch_words = a.in_h * a.pitch;
  uint16_t* off = reinterpret_cast<uint16_t*>(tile + (size_t)a.d.C * ch_words);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  fill_offsets(a, off, ch_words, threadIdx.x, THREADS);
  const int64_t total_tiles = (int64_t)a.tiles_h * a.tiles_w * a.d.N;
  for (int64_t tile_id = blockIdx.x; tile_id < total_tiles; tile_id += gridDim.x) {
    const TileCoord t = tile_coord(a, tile_id);
    __syncthreads();
    load_tile<false>(a, a.x + (int64_t)t.img * a.d.C * a.d.H * a.d.W, t.h0, t.w0, tile, ch_words, threadIdx.x, THREADS);
    __syncthreads();
    for (int p = warp; p < t.th * t.tw; p += kWarpsPerCta) {
      const int lh = p / t.tw, lw = p % t.tw;
      const float* origin = tile + lh * a.d.stride_h * a.pitch + lw * a.d.stride_w;
      auto value = [origin, off](int i) { return origin[off[i]]; };
      const int64_t pi = ((int64_t)t.img * a.Ho + (t.ho0 + lh)) * a.Wo + (t.wo0 + lw);
      warp_sign_row(value, a.n, a.ldp, lane, a.pK + pi, a.pgamma + pi, a.pdelta + pi,
                    a.pflags ? a.pflags + pi : nullptr, a.pmask + pi * (int64_t)a.ldp);
    }
  }
}

__global__ void __launch_bounds__(256) sign_rows_kernel(const float* __restrict__ values, int64_t rows, int32_t n,
                                                        int64_t ld_values, int32_t* K, float* alpha, float* beta,
                                                        uint32_t* mask, int32_t ld_mask, uint32_t* flags) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t row = warp0; row < rows; row += nwarps) {
    const float* v = values + row * ld_values;
    auto value = [v](int i) { return __ldg(v + i); };
    warp_sign_row(value, n, ld_mask, lane, K + row, alpha + row, beta + row, flags ? flags + row : nullptr,
                  mask + row * (int64_t)ld_mask);
  }
}

cudaError_t launch_sign_rows(const float* values, int64_t rows, int32_t n, int64_t ld_values, int32_t* K, float* alpha,
                             float* beta, uint32_t* mask, int32_t ld_mask, uint32_t* flags, cudaStream_t stream) {
  int64_t blocks = (rows + 7) / 8;
  if (blocks > sm_count() * 16) blocks = sm_count() * 16;
  sign_rows_kernel<<<(unsigned)blocks, 256, 0, stream>>>(values, rows, n, ld_values, K, alpha, beta, mask, ld_mask,
                                                        flags);
  return cudaGetLastError();
}

// 0: by tile density (default), 1: sort-based coders only, 2: histogram-pruned coder wherever it applies.
static std::atomic<int> g_patch_coder_mode{0};

int patch_coder_mode() { return g_patch_coder_mode.load(std::memory_order_relaxed); }
void set_patch_coder_mode(int mode) { g_patch_coder_mode.store(mode, std::memory_order_relaxed); }

// Tile shapes tried, largest first.
static const int kTileShapes[][2] = {{8, 8}, {4, 8}, {4, 4}, {2, 4}, {2, 2}, {1, 2}, {1, 1}};

static void set_tile(const dab_conv_desc& d, int Ho, int Wo, const int (&sh)[2], PatchArgs* a) {
  int TH = sh[0] < Ho ? sh[0] : Ho, TW = sh[1] < Wo ? sh[1] : Wo;
  int in_h = (TH - 1) * d.stride_h + d.kh, in_w = (TW - 1) * d.stride_w + d.kw;
  a->TH = TH; a->TW = TW; a->in_h = in_h; a->in_w = in_w;
  a->pitch = in_w | 1;  // odd pitch spreads the rows of a patch over the banks
  a->tiles_h = (Ho + TH - 1) / TH; a->tiles_w = (Wo + TW - 1) / TW;
  const uint64_t pc = (uint64_t)in_h * in_w, two32 = 0x100000000ull;
  a->magic_per_ch = pc > 1 ? (uint32_t)((two32 + pc - 1) / pc) : 0u;
  a->magic_in_w = in_w > 1 ? (uint32_t)((two32 + (uint64_t)in_w - 1) / (uint64_t)in_w) : 0u;
}

// Picks the tile and launches.  A shape is admissible if its staged input fits and it leaves 16 to 24 warps
// resident per SM (shared memory is the limit); `groups` = patches a CTA codes at a time.  Among the admissible
// shapes the largest one that still gives two CTAs per SM of work is taken (large layers: least halo re-reading);
// a small layer, which cannot fill the GPU with large tiles, gets the smallest shape that keeps all groups of a
// CTA busy (most CTAs, shortest critical path).  If nothing is admissible the shape with the most resident CTAs wins.
template <typename Kernel>
static cudaError_t launch_patches(Kernel kern, PatchArgs& a, size_t fixed_bytes, int threads, int groups,
                                  cudaStream_t stream, bool shape_only = false) {
  const size_t sm_bytes = 228 * 1024, cta_reserve = 1024, cta_limit = 227 * 1024;
  // resident warps per SM a shape must leave room for: measured best is 24 for one or two warps per patch (their
  // tile loads overlap other CTAs' sorting), 16 for larger groups (fewer, larger tiles matter more)
  const int want_warps = groups >= 4 ? 24 : 16;
  const int want_ctas = (want_warps * 32 + threads - 1) / threads;
  const int64_t want_tiles = 2 * sm_count();
  int best = -1, best_ctas = 0, small = -1;
  size_t best_smem = 0, small_smem = 0;
  bool settled = false;
  for (int i = 0; i < (int)(sizeof(kTileShapes) / sizeof(kTileShapes[0])) && !settled; ++i) {
    if (a.tile_shape >= 0 && i != a.tile_shape) continue;
    PatchArgs t = a;
    set_tile(a.d, a.Ho, a.Wo, kTileShapes[i], &t);
    size_t tile_words = (size_t)a.d.C * t.in_h * t.pitch;
    if (tile_words > 65535) continue;  // offsets are 16-bit
    size_t smem = fixed_bytes + tile_words * sizeof(float) + sizeof(uint16_t) * a.n + 16;
    if (smem > cta_limit) continue;
    int ctas = (int)(sm_bytes / (smem + cta_reserve));
    if (ctas > 2048 / threads) ctas = 2048 / threads;
    if (ctas > best_ctas) { best = i; best_ctas = ctas; best_smem = smem; }
    if (ctas >= want_ctas) {
      const int64_t tiles = (int64_t)t.tiles_h * t.tiles_w * a.d.N;
      const bool busy = t.TH * t.TW >= groups;  // every group of the CTA has a patch
      if ((tiles >= want_tiles && busy) || a.tile_shape >= 0) { best = i; best_smem = smem; settled = true; }
      else if (busy || small < 0) { small = i; small_smem = smem; }
    }
  }
  if (!settled && small >= 0) { best = small; best_smem = small_smem; }
  if (best < 0) return cudaErrorInvalidValue;
  a.tile_shape = best;
  set_tile(a.d, a.Ho, a.Wo, kTileShapes[best], &a);
  if (shape_only) return cudaSuccess;  // the caller wanted the tile this kernel would take
  cudaError_t e = ensure_dynamic_smem(kern, best_smem);
  if (e != cudaSuccess) return e;
  int64_t tiles = (int64_t)a.tiles_h * a.tiles_w * a.d.N;
  int64_t blocks = tiles < sm_count() * 8 ? tiles : sm_count() * 8;
  kern<<<(unsigned)blocks, threads, best_smem, stream>>>(a);
  return cudaGetLastError();
}

template <int R, bool kFull>
static cudaError_t launch_patches_warp(PatchArgs& a, cudaStream_t stream) {
  size_t fixed = sizeof(double) * rcp_table_slots(a.n) + sizeof(uint32_t) * 32 * R * kWarpsPerCta;
  return launch_patches(binarize_patches_warp_kernel<R, kFull>, a, fixed, kWarpsPerCta * 32, kWarpsPerCta, stream);
}

template <int W, int WARPS, int R, bool kFull, bool kTable>
static cudaError_t launch_patches_group(PatchArgs& a, cudaStream_t stream, bool shape_only = false) {
  constexpr int G = WARPS / W;
  a.scratch_words = scratch_words_for(a.n, W);
  size_t fixed = (kTable ? sizeof(double) * rcp_table_slots(a.n) : 0) + sizeof(GroupShared) * G +
                 sizeof(uint32_t) * (size_t)a.scratch_words * G;
  return launch_patches(binarize_patches_group_kernel<W, WARPS, R, kFull, kTable>, a, fixed, WARPS * 32, G, stream,
                        shape_only);
}

template <int BPL>
static cudaError_t launch_patches_hist(PatchArgs& a, cudaStream_t stream) {
  // beyond the group kernel's tile: one more word per channel (odd channel pitch) and the window offsets
  size_t fixed = sizeof(double) * rcp_table_slots(a.n) + sizeof(int2) * 32 * BPL * kWarpsPerCta +
                 sizeof(uint32_t) * hist_cap(BPL) * kWarpsPerCta + sizeof(float) * a.d.C +
                 sizeof(uint16_t) * (size_t)(a.d.kh * a.d.kw + 2);
  if (a.d.kh * a.d.kw == 9)
    return launch_patches(binarize_patches_hist_kernel<BPL, 9>, a, fixed, kWarpsPerCta * 32, kWarpsPerCta, stream);
  return launch_patches(binarize_patches_hist_kernel<BPL, 0>, a, fixed, kWarpsPerCta * 32, kWarpsPerCta, stream);
}

// Buckets by patch length: enough of them that the few that survive hold well under the 256 or 1024 values the exact search takes.
static cudaError_t launch_hist_for(PatchArgs& a, cudaStream_t stream) {
  if (a.n < 1024) return launch_patches_hist<2>(a, stream);
  if (a.n < 4096) return launch_patches_hist<4>(a, stream);
  return launch_patches_hist<8>(a, stream);
}

// The group kernel that codes patches of n > 256 values (the sort-based coder for these lengths, and the one
// that takes the tiles the other coders mark).
static cudaError_t launch_group_for(PatchArgs& a, cudaStream_t stream, bool shape_only) {
  if (a.n <= 576) return launch_patches_group<4, 8, 5, false, true>(a, stream, shape_only);
  if (a.n <= 1024) return launch_patches_group<2, 8, 16, false, true>(a, stream, shape_only);
  if (a.n == 1152) return launch_patches_group<2, 8, 18, true, true>(a, stream, shape_only);
  if (a.n <= 2048) return launch_patches_group<4, 8, 16, false, true>(a, stream, shape_only);
  if (a.n == 2304) return launch_patches_group<4, 8, 18, true, true>(a, stream, shape_only);
  if (a.n <= 4096) return launch_patches_group<8, 16, 16, false, true>(a, stream, shape_only);
  if (a.n == 4608) return launch_patches_group<8, 16, 18, true, true>(a, stream, shape_only);
  if (a.n <= 8192) return launch_patches_group<16, 16, 16, false, true>(a, stream, shape_only);
  if (a.n == 9216) return launch_patches_group<16, 16, 18, true, false>(a, stream, shape_only);
  return launch_patches_group<16, 16, 32, false, false>(a, stream, shape_only);
}

cudaError_t launch_sign_patches(const dab_conv_desc& d, int32_t Ho, int32_t Wo, const float* x, int32_t* pK,
                                float* pgamma, float* pdelta, uint32_t* pmask, int32_t ldp, uint32_t* pflags,
                                cudaStream_t stream) {
  PatchArgs a;
  a.d = d; a.Ho = Ho; a.Wo = Wo; a.n = d.C * d.kh * d.kw;
  a.scratch_words = 0;
  a.defer_dense = 0; a.marked_only = 0; a.tile_shape = -1;
  a.x = x; a.pK = pK; a.pgamma = pgamma; a.pdelta = pdelta; a.pflags = pflags; a.pmask = pmask; a.ldp = ldp;
  return launch_patches(sign_patches_kernel, a, 0, kWarpsPerCta * 32, kWarpsPerCta, stream);
}

cudaError_t launch_binarize_patches(const dab_conv_desc& d, int32_t Ho, int32_t Wo, const float* x, int32_t* pK,
                                    float* pgamma, float* pdelta, uint32_t* pmask, int32_t ldp, uint32_t* pflags,
                                    cudaStream_t stream) {
  PatchArgs a;
  a.d = d; a.Ho = Ho; a.Wo = Wo; a.n = d.C * d.kh * d.kw;
  a.scratch_words = 0;
  a.defer_dense = 0; a.marked_only = 0; a.tile_shape = -1;
  a.x = x; a.pK = pK; a.pgamma = pgamma; a.pdelta = pdelta; a.pflags = pflags; a.pmask = pmask; a.ldp = ldp;
  a.dense_num = 1; a.dense_den = 0;  // no tile counts as dense unless a chain below says so
  if (a.n <= 256) return launch_patches_warp<8, false>(a, stream);
  const int mode = patch_coder_mode();
  cudaError_t e;
  // The pixel-histogram coder shares work between overlapping patches: it is the default wherever a patch spans
  // several pixels and the layer has enough patches to fill the device with its tiles (measured: from about a
  // thousand patches).
  const bool pixel_default = d.kh * d.kw >= 4 && (int64_t)d.N * Ho * Wo >= 1024;
  if (mode == 3 || (mode == 0 && pixel_default)) {
    bool applicable = false;
    e = launch_binarize_patches_pixhist(d, Ho, Wo, x, pK, pgamma, pdelta, pmask, ldp, pflags, stream, &applicable);
    if (e != cudaSuccess || applicable) return e;
  }
  if (mode == 1 || a.n > 8192) {
    // Sort-based coders only.  The patch lengths of the common 3x3 layers (576 values per warp) have variants
    // without bounds tests whose group size suits rows that are at least half zeros.
    if (a.n <= 576) {
      // first the one-warp kernel on the tiles it suits, then four warps per patch on the tiles it marked as dense
      // (expected non-zeros per patch = density of the staged region * n > 256)
      a.defer_dense = 1; a.dense_num = 256; a.dense_den = a.n;
      e = a.n == 576 ? launch_patches_warp<18, true>(a, stream) : launch_patches_warp<18, false>(a, stream);
      if (e != cudaSuccess) return e;
      a.defer_dense = 0; a.marked_only = 1;  // a.tile_shape now holds the first kernel's tile
      return launch_group_for(a, stream, false);
    }
    return launch_group_for(a, stream, false);
  }
  // The histogram-pruned coder runs on the tile shape of the group kernel, which ends every chain by taking the
  // tiles nobody else settled.  Its 16-bit offsets must reach the whole (odd-pitched) tile.
  if ((e = launch_group_for(a, stream, /*shape_only=*/true)) != cudaSuccess) return e;
  const bool hist_fits = (size_t)a.d.C * ((a.in_h * a.pitch) | 1) <= 65535;
  if (mode == 2) {  // everything through the histogram coder
    if (hist_fits) {
      e = launch_hist_for(a, stream);
      if (e != cudaSuccess) return e;
      a.marked_only = 1;
    }
    return launch_group_for(a, stream, false);
  }
  // By density: the sort-based coder of this length takes the sparse tiles and marks the dense ones; the
  // histogram coder, whose cost does not grow with the number of non-zero values, takes those; the group kernel
  // takes what that one leaves.  Tiles count as dense above 256 / n (patches of up to 576 values) or 45 %
  // non-zero values: about the density from which the sorting kernels need more than 8 keys per thread.
  if (!hist_fits) {
    a.tile_shape = -1;
    return launch_group_for(a, stream, false);
  }
  a.defer_dense = 1;
  if (a.n <= 576) {
    a.dense_num = 256; a.dense_den = a.n;  // expected non-zeros per patch above the 256 one warp sorts with 8 keys per lane
    a.tile_shape = -1;  // the one-warp kernel picks its own tile; the two kernels after it take it over
    e = a.n == 576 ? launch_patches_warp<18, true>(a, stream) : launch_patches_warp<18, false>(a, stream);
  } else {
    a.dense_num = 45; a.dense_den = 100;
    e = launch_group_for(a, stream, false);
  }
  if (e != cudaSuccess) return e;
  a.defer_dense = 0; a.marked_only = 1;
  if ((size_t)a.d.C * ((a.in_h * a.pitch) | 1) <= 65535) {  // (the first kernel may have taken another tile)
    e = launch_hist_for(a, stream);
    if (e != cudaSuccess) return e;
  }
  return launch_group_for(a, stream, false);
}

}  // namespace dab

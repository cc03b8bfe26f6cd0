// Patch coder that shares work between overlapping patches (Section 4.1 / Algorithm 1 per patch; Section 4.3.1
// asks for all rows of a layer to be handled as one batch).
//
// A patch is the union of kh*kw pixels (a pixel = the C channel values at one input position) and every pixel
// belongs to up to kh*kw patches, so whatever can be prepared per pixel is prepared once per tile:
//   per tile   the non-zero values of every staged pixel are counted into B buckets of equal width (a power of
//              two, so that bucket bounds are exact), counting-sorted by bucket into a per-pixel list of channel
//              indices, and the per-pixel cumulative (count, fp64 sum) per bucket are tabulated;
//   per patch  (one warp) the cumulative tables of its kh*kw pixels are added: that gives, at every bucket edge, the
//              split size s and the prefix sum P of the patch, exactly.  The objective D = P^2/s + (T-P)^2/(n-s) is
//              jointly convex in (s, P); inside a bucket the pair (s, P) stays within a parallelogram fixed by the
//              bucket's count, sum and value bounds, so D is bounded there by its values at the parallelogram's
//              corners.  Buckets whose bound stays below the best edge value cannot hold the maximum.  The few
//              values of the buckets that can (the "hull") are gathered from the per-pixel lists, sorted and
//              searched by the exact evaluator of rowcode.cuh with the exact counts and sums below and above
//              them as its base.  The mask is a threshold compare over the patch.
// The bounds are evaluated in fp32 from fp64 inputs with a relative margin of 2e-5 (see prune_margin); a patch the
// search does not settle (a hull above the cap, a degenerate row, an extreme dynamic range, a NaN or infinity in
// the tile) is marked K = kRowMark and coded by the full-sort kernel that follows on the stream.
#include <cmath>

#include "histcode.cuh"
#include "rowcode.cuh"

#ifndef DAB_PIX_UNROLL
#define DAB_PIX_UNROLL 4   // channels of one pixel a warp keeps in flight in the per-tile passes
#endif

namespace dab {

namespace {

constexpr int kPixUnroll = DAB_PIX_UNROLL;

constexpr int kFixWarps = 8;      // warps of the kernel that sorts the marked patches
constexpr int kFixThreads = kFixWarps * 32;
constexpr int kHullCap = 256;        // values the exact search takes at most from the per-warp scratch array (8 per lane)
constexpr int kHullCapRegs = 1024;   // the same when the hull goes straight into registers (3 x 3 windows; 32 per lane)

struct PixArgs {
  dab_conv_desc d;
  int32_t Ho, Wo, n;
  int32_t TH, TW;           // output positions per tile
  int32_t in_h, in_w, pix;  // staged rows, columns and pixels per tile
  int32_t ch_words;         // words per staged channel: pix | 1
  int32_t tiles_h, tiles_w;
  const float* x;
  int32_t* pK;
  float* pgamma;
  float* pdelta;
  uint32_t* pflags;  // may be null
  uint32_t* pmask;
  int32_t ldp;
};

// Patches of the call: the extent of pK, pgamma, pdelta and pflags (and, times ldp, of pmask).
__device__ __forceinline__ int64_t patch_count(const PixArgs& a) { return (int64_t)a.d.N * a.Ho * a.Wo; }

// Bucket grid of a tile: buckets of equal width within each octave of magnitude, 2^m per octave.  The bucket of a
// value is the bit pattern of its magnitude shifted right by 23 - m, minus a base that puts the tile's largest
// magnitude into the last bucket of its side; everything below the resolved octaves shares the bucket next to zero.
// The edges are the floats with those leading bits, so membership is exact.
//   One sign only (post-ReLU activations): all B buckets over the top B / 2^m = 4 octaves.  The best split of such
//   rows lies among the larger values.
//   Both signs: B/2 buckets on either side of zero over the top 8 octaves.  Such rows often split near zero, where
//   this grid is finest in absolute terms, and a heavy tail costs it one bucket per half octave instead of
//   stretching every bucket.
// Relative resolution is what the search needs: buckets of one width over the whole range spend most of them where
// values are rare, and one outlier in the tile widens them all.  (Kernels compiled without kOctaves use that
// equal-width grid, bucket(v) = floor(v * 2^k) + B0 with k the largest exponent that fits the range; none is by
// default.)
struct PixQuant {
  int shift;  // per-octave grid: 23 - m; 0: equal widths
  int p;      // per-octave grid: the base of the shifted bit pattern; equal widths: the bits of 2^k as a float
  int B0;     // first bucket of the positive values (0: none negative, B: none positive, B/2: both signs)
  bool ok;    // false: magnitudes outside [2^-40, 2^40]; the tile goes to the sorting kernel
};

#ifndef DAB_PIX_COST_PATCH
#define DAB_PIX_COST_PATCH 5000.0  // cost model of the tile choice: cycles per patch, ...
#define DAB_PIX_COST_VALUE 5.0     // ... plus this per value of the patch (a staged value of the tile costs 4.6)
#endif
#ifndef DAB_PIX_N2
#define DAB_PIX_N2 2048  // rows shorter than this take 32 buckets, ...
#define DAB_PIX_N4 4096  // ... than this 64, longer ones 128
#endif
#ifndef DAB_PIX_OCTAVES_UPTO_BPL
#define DAB_PIX_OCTAVES_UPTO_BPL 8  // kernels with this many buckets per lane or fewer use the per-octave grid
#endif
#ifndef DAB_PIX_OCTAVES_LOG2
#define DAB_PIX_OCTAVES_LOG2 2        // the per-octave grid resolves the top 2^2 = 4 octaves of a one-signed tile's magnitudes
#endif
#ifndef DAB_PIX_OCTAVES_MIXED_LOG2
#define DAB_PIX_OCTAVES_MIXED_LOG2 3  // and the top 2^3 = 8 octaves on either side of zero of a tile with both signs
#endif

template <bool kOctaves>
__device__ __forceinline__ PixQuant make_pix_quant(uint32_t kmin, uint32_t kmax, int LOG2B) {
  PixQuant q;
  const float lo = key_value(kmin), hi = key_value(kmax);
  const float A = fmaxf(fabsf(lo), fabsf(hi));
  const int e = (int)((__float_as_uint(A) >> 23) & 255u) - 127;  // A in [2^e, 2^(e+1))
  q.ok = e >= -40 && e <= 40;
  const bool mixed = lo < 0.0f && hi > 0.0f;
  const int k = (mixed ? LOG2B - 1 : LOG2B) - e - 1;
  const int kc = min(max(k, -100), 100);
  q.B0 = lo > 0.0f ? 0 : (hi < 0.0f ? (1 << LOG2B) : (1 << (LOG2B - 1)));
  q.shift = 0;
  q.p = (kc + 127) << 23;
  if (kOctaves) {  // 2^m buckets per octave; e >= -40 keeps the base positive
    // one sign: all B buckets over the top four octaves; both signs: B/2 per sign over the top eight
    const int side = mixed ? (1 << (LOG2B - 1)) : (1 << LOG2B);
    q.shift = 23 - (mixed ? LOG2B - 1 - DAB_PIX_OCTAVES_MIXED_LOG2 : LOG2B - DAB_PIX_OCTAVES_LOG2);
    q.p = (int)(__float_as_uint(A) >> q.shift) - (side - 1);
  }
  return q;
}

// (A negative value so small that the product rounds to -0.0 still belongs below zero.)
template <bool kOctaves>
__device__ __forceinline__ int pix_bucket(float v, const PixQuant& q, int B) {
  if (kOctaves && q.shift) {  // magnitudes ascend with the bucket on the positive side, descend on the negative one
    const int side = (q.B0 > 0 && q.B0 < B) ? B >> 1 : B;  // buckets per sign
    const int i = min(max((int)((__float_as_uint(v) & 0x7FFFFFFFu) >> q.shift) - q.p, 0), side - 1);
    return v < 0.0f ? q.B0 - 1 - i : q.B0 + i;
  }
  int f = __float2int_rd(v * __int_as_float(q.p));
  if (v < 0.0f) f = min(f, -1);
  return min(max(f + q.B0, 0), B - 1);
}

// Values bucket b can hold, [vlo, vhi), and the reciprocal of its width (exact for every bucket but the one next
// to zero of the per-octave grid, where it is good to 2e-14 relative).
template <bool kOctaves>
__device__ __forceinline__ void pix_bucket_range(const PixQuant& q, int b, int B, double& vlo, double& vhi,
                                                 double& inv_width) {
  if (kOctaves && q.shift) {
    const bool negative = b < q.B0;
    const int i = negative ? q.B0 - 1 - b : b - q.B0;
    const float lo = i ? __uint_as_float((uint32_t)(i + q.p) << q.shift) : 0.0f;
    const float hi = __uint_as_float((uint32_t)(i + 1 + q.p) << q.shift);
    vlo = negative ? -(double)hi : (double)lo;
    vhi = negative ? -(double)lo : (double)hi;
    // hi - lo = 2^(exponent of lo - m) with m = 23 - shift: its reciprocal by exponent arithmetic; next to zero 1 / hi
    const int biased = (int)((uint32_t)(i + q.p) >> (23 - q.shift));  // exponent field of lo
    const double r = i ? (double)__int_as_float((254 + (23 - q.shift) - biased) << 23) : (double)__fdividef(1.0f, hi);
    // one Newton step: leaves the exact reciprocals as they are and takes 1 / hi from 2 ulp of fp32 to 2e-14 relative
    inv_width = __dmul_rn(r, __dsub_rn(2.0, __dmul_rn(vhi - vlo, r)));
    return;
  }
  const double width = (double)__int_as_float((254 << 23) - q.p);  // q.p holds the bits of 2^k: 2^-k, exact
  vlo = (double)(b - q.B0) * width;
  vhi = vlo + width;
  inv_width = (double)__int_as_float(q.p);
}

// Objective in fp32 from fp64 coordinates: every input is rounded once (relative 2^-24), both terms are
// non-negative, the two quotients are good to 2 ulp: the result is within 1e-6 relative of the exact value for
// results inside the normal fp32 range.  s = 0 and s = n stand for the limits (P = 0 resp. P = T there).
__device__ __forceinline__ float objective_bound(double s, double P, double T, double nd) {
  const float Pf = (float)P, Qf = (float)(T - P), sf = (float)s, rf = (float)(nd - s);
  const float a = sf > 0.0f ? __fdividef(Pf * Pf, sf) : 0.0f;
  const float b = rf > 0.0f ? __fdividef(Qf * Qf, rf) : 0.0f;
  return a + b;
}

// A candidate is kept if its fp32 value reaches best * prune_margin: with both sides within 1e-6 of their exact
// values, anything whose exact bound reaches the exact best edge value is kept.
constexpr float prune_margin = 0.99998f;

template <int E, bool kTable>
__device__ __noinline__ RowResult pix_sort_select(const uint32_t* scratch, int m, int z, int n, int lane,
                                                  const double* rcp, const SplitBase base) {
  uint32_t r[E];
#pragma unroll
  for (int j = 0; j < E; ++j) {
    const int idx = j * 32 + lane;
    r[j] = idx < m ? order_key(__uint_as_float(scratch[idx])) : kPadKey;  // the gather stored raw bits
  }
  group_sort<1, E>(r, lane, nullptr, 0);
  return group_select<1, E, kTable, true>(r, m, z, n, lane, nullptr, 0, rcp, base);
}

// The same with the hull taken straight from the ordered lists of the window's pixels into registers.  Lane rs of the
// first 16 holds, for pixel rs of the window, the pixel (my_pq), where its part of the hull starts in its list
// (my_st) and how many values of all the parts come before it (excl; lanes beyond the window hold the total).
template <int E, bool kTable, typename ListT>
__device__ __noinline__ RowResult pix_gather_sort_select(const float* tile, const ListT* list, int C, int chw, int excl,
                                                         int my_st, int my_pq, int npix, int m, int z, int n, int lane,
                                                         const double* rcp, const SplitBase base) {
  uint32_t r[E];
#pragma unroll
  for (int j = 0; j < E; ++j) {
    const int i = j * 32 + lane;
    int rs = 0;  // the last pixel whose part starts at or before i (parts after it that start there are empty)
#pragma unroll
    for (int step = 8; step >= 1; step >>= 1) {
      const int cand = rs + step;
      const int o = __shfl_sync(0xFFFFFFFFu, excl, cand & 15);
      if (cand < npix && i >= o) rs = cand;
    }
    const int o = __shfl_sync(0xFFFFFFFFu, excl, rs);
    const int st = __shfl_sync(0xFFFFFFFFu, my_st, rs);
    const int pq = __shfl_sync(0xFFFFFFFFu, my_pq, rs);
    r[j] = kPadKey;
    if (i < m) r[j] = order_key(tile[(int)list[pq * C + st + (i - o)] * chw + pq]);
  }
  group_sort<1, E>(r, lane, nullptr, 0);
  return group_select<1, E, kTable, true>(r, m, z, n, lane, nullptr, 0, rcp, base);
}

// WARPS: warps per CTA; BPL: buckets per lane (B = 32 BPL); KHW: kh*kw when it is 9 (window loops unrolled, masks
// assembled per channel), 0 for any other window; ListT: type of a channel index; kTable: reciprocal table in
// shared memory.
template <int WARPS, int MINB, int BPL, int KHW, typename ListT, bool kTable>
__global__ void __launch_bounds__(WARPS * 32, MINB) binarize_patches_pixhist_kernel(const PixArgs a) {
  constexpr int THREADS = WARPS * 32;
  constexpr int B = 32 * BPL;
  constexpr bool kOctaves = BPL <= DAB_PIX_OCTAVES_UPTO_BPL;  // single-signed tiles take the per-octave grid
  constexpr int LOG2B = BPL == 1 ? 5 : BPL == 2 ? 6 : BPL == 4 ? 7 : 8;
  constexpr int SS = B + 1;  // table row stride: odd, so that one thread per pixel walks its row without conflicts
  constexpr int KMAX = KHW ? KHW : 1;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* rcp = reinterpret_cast<double*>(smem_raw);
  double* sumc = rcp + (kTable ? rcp_table_slots(a.n) : 0);                 // [pix][SS] cumulative sums
  int* cntc = reinterpret_cast<int*>(sumc + (size_t)a.pix * SS);            // [pix][SS] cumulative counts
  float* tile = reinterpret_cast<float*>(cntc + (size_t)a.pix * SS);        // [C][ch_words]
  uint32_t* scratch_all = reinterpret_cast<uint32_t*>(tile + (size_t)a.d.C * a.ch_words);  // KHW == 0 only
  uint32_t* pinfo = scratch_all + (KHW ? 0 : WARPS * kHullCap);             // [64] per patch of the tile: window origin, (lh, lw)
  int* poff = reinterpret_cast<int*>(pinfo + 64);                           // [pix] offset of the pixel in its channel plane, -1: outside the image
  uint16_t* win = reinterpret_cast<uint16_t*>(poff + a.pix);                  // [kh*kw] pixel offsets of the window
  uint16_t* off = win + ((a.d.kh * a.d.kw + 1) & ~1);                       // [n] element offsets (KHW == 0 only)
  ListT* list = reinterpret_cast<ListT*>(off + (KHW ? 0 : ((a.n + 1) & ~1)));  // [pix][C] channels by bucket

  __shared__ uint32_t s_kmin, s_kmax;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int C = a.d.C, pixn = a.pix, chw = a.ch_words, khw = a.d.kh * a.d.kw;
  uint32_t* scratch = scratch_all + warp * kHullCap;
  if (kTable) fill_reciprocals(rcp, a.n, threadIdx.x, THREADS);
  for (int rs = threadIdx.x; rs < khw; rs += THREADS) win[rs] = (uint16_t)((rs / a.d.kw) * a.in_w + rs % a.d.kw);
  if (!KHW) {
    for (int i = threadIdx.x; i < a.n; i += THREADS) {
      const int c = i / khw, rs = i % khw;
      off[i] = (uint16_t)(c * chw + (rs / a.d.kw) * a.in_w + rs % a.d.kw);
    }
  }
  __syncthreads();
  const int in_w = a.in_w;
  // pixel offset of window position rs (3 x 3 windows: KHW == 9); rs is a compile-time constant wherever this is used
  auto wofs = [in_w](int rs) { return (rs / 3) * in_w + rs % 3; };
  // runs of lanes whose 9-bit fields start in the same mask word (word = 9 * lane / 32), see the mask assembly
  const int my_word = (lane * 9) >> 5;
  uint32_t run_next = 0u;  // bit d-1: lane + d belongs to this lane's run
#pragma unroll
  for (int d = 1; d <= 3; ++d) run_next |= (lane + d < 32 && (((lane + d) * 9) >> 5) == my_word) ? (1u << (d - 1)) : 0u;
  const int first_of_word = (min(lane, 8) * 32 + 8) / 9;                   // first lane whose field starts in word `lane`
  const int first_of_prev = (max(min(lane, 8) - 1, 0) * 32 + 8) / 9;       // the same for the word before
  const double nd = (double)a.n;
  const int rounds = (a.n + 31) >> 5;

  const int64_t tiles_per_img = (int64_t)a.tiles_h * a.tiles_w;
  const int64_t total_tiles = tiles_per_img * a.d.N;
  for (int64_t tile_id = blockIdx.x; tile_id < total_tiles; tile_id += gridDim.x) {
    const int img = (int)(tile_id / tiles_per_img);
    const int trem = (int)(tile_id % tiles_per_img);
    const int ho0 = (trem / a.tiles_w) * a.TH, wo0 = (trem % a.tiles_w) * a.TW;
    const int h0 = ho0 * a.d.stride_h - a.d.pad_h, w0 = wo0 * a.d.stride_w - a.d.pad_w;
    const int th = min(a.TH, a.Ho - ho0), tw = min(a.TW, a.Wo - wo0);
    const int npatch = th * tw;
    const int64_t tile_base = ((int64_t)img * a.Ho + ho0) * a.Wo + wo0;  // index of the tile's first patch
    __syncthreads();  // the previous tile is no longer read
    if (threadIdx.x == 0) { s_kmin = kPadKey; s_kmax = 0u; }
    for (int i = threadIdx.x; i < pixn * SS; i += THREADS) { cntc[i] = 0; sumc[i] = 0.0; }
    if (threadIdx.x < npatch) {
      const int lh = threadIdx.x / tw, lw = threadIdx.x % tw;
      pinfo[threadIdx.x] = (uint32_t)(lh * a.d.stride_h * a.in_w + lw * a.d.stride_w) | ((uint32_t)lw << 16) | ((uint32_t)lh << 24);
    }
    for (int p = threadIdx.x; p < pixn; p += THREADS) {
      const int r = p / a.in_w, s = p - r * a.in_w;
      const int h = h0 + r, w = w0 + s;
      poff[p] = ((unsigned)h < (unsigned)a.d.H && (unsigned)w < (unsigned)a.d.W) ? h * a.d.W + w : -1;
    }
    __syncthreads();
    {  // stage the tile: a warp per channel, a lane per pixel; asynchronous 4-byte copies, zeros outside the image
      const float* ximg = a.x + (int64_t)img * C * a.d.H * a.d.W;
      const int plane = a.d.H * a.d.W;
      for (int p = lane; p < pixn; p += 32) {
        const int o = poff[p];
        if (o >= 0) {
          const unsigned saddr = (unsigned)__cvta_generic_to_shared(tile + p);
#pragma unroll kPixUnroll
          for (int c = warp; c < C; c += WARPS)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(saddr + 4u * (unsigned)(c * chw)),
                         "l"(ximg + DAB_IDX(o + (int64_t)c * plane, (int64_t)C * plane)) : "memory");
        } else {
          for (int c = warp; c < C; c += WARPS) tile[c * chw + p] = 0.0f;
        }
      }
      asm volatile("cp.async.wait_all;" ::: "memory");
    }
    __syncthreads();
    {  // range of the non-zero values (-0.0 counts as zero everywhere below: every use is a comparison)
      uint32_t kmin = kPadKey, kmax = 0u;
      for (int p = lane; p < pixn; p += 32) {
#pragma unroll kPixUnroll
        for (int c = warp; c < C; c += WARPS) {
          const float v = tile[c * chw + p];
          const uint32_t key = order_key(v);
          const bool nz = v != 0.0f;  // NaN compares unequal: counted, and seen as non-finite below
          kmin = min(kmin, nz ? key : kPadKey);
          kmax = max(kmax, nz ? key : 0u);
        }
      }
      kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
      kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
      if (lane == 0 && kmin <= kmax) {
        atomicMin(&s_kmin, kmin);
        atomicMax(&s_kmax, kmax);
      }
    }
    __syncthreads();
    const uint32_t tkmin = s_kmin, tkmax = s_kmax;
    const bool any_nonzero = tkmin <= tkmax;
    PixQuant qz = make_pix_quant<kOctaves>(any_nonzero ? tkmin : kZeroKey + 1u, any_nonzero ? tkmax : kZeroKey + 1u, LOG2B);
    if (any_nonzero && (key_range_nonfinite(tkmin, tkmax) || !qz.ok)) {
      // every patch of the tile is left to the sorting kernel
      for (int p = threadIdx.x; p < npatch; p += THREADS) {
        const int64_t pi = tile_base + (int64_t)(p / tw) * a.Wo + p % tw;
        if (DAB_IN_BOUNDS(pi, patch_count(a))) a.pK[pi] = kRowMark;
      }
      continue;
    }
    // ---- per pixel: count and fp64 sum per bucket ----
    for (int p = lane; p < pixn; p += 32) {
#pragma unroll kPixUnroll
      for (int c = warp; c < C; c += WARPS) {
        const float v = tile[c * chw + p];
        if (v != 0.0f) {
          const int slot = p * SS + pix_bucket<kOctaves>(v, qz, B);
          atomicAdd(&cntc[slot], 1);
          atomicAdd(&sumc[slot], (double)v);
        }
      }
    }
    __syncthreads();
    // ---- per pixel (one thread each): exclusive scan of the counts, inclusive scan of the sums ----
    for (int p = threadIdx.x; p < pixn; p += THREADS) {
      int run = 0;
      double runs = 0.0;
      int* row = cntc + p * SS;
      double* srow = sumc + p * SS;
      for (int b = 0; b < B; ++b) {
        const int c = row[b];
        row[b] = run;
        run += c;
        runs = __dadd_rn(runs, srow[b]);
        srow[b] = runs;
      }
    }
    __syncthreads();
    // ---- per pixel: channel indices ordered by bucket; the cursors end as inclusive cumulative counts ----
    for (int p = lane; p < pixn; p += 32) {
#pragma unroll kPixUnroll
      for (int c = warp; c < C; c += WARPS) {
        const float v = tile[c * chw + p];
        if (v != 0.0f) {
          const int pos = atomicAdd(&cntc[p * SS + pix_bucket<kOctaves>(v, qz, B)], 1);
          list[p * C + pos] = (ListT)c;
        }
      }
    }
    __syncthreads();

    // ---- patches: one warp each ----
    for (int p = warp; p < npatch; p += WARPS) {
      const uint32_t info = pinfo[p];
      const int pix0 = (int)(info & 0xFFFFu);  // first pixel of the window
      const int64_t pi = tile_base + (int64_t)(info >> 24) * a.Wo + ((info >> 16) & 255u);
      uint32_t* mrow = a.pmask + pi * (int64_t)a.ldp;

      // cumulative count and sum of the patch at the upper edge of this lane's buckets (bucket j*32 + lane)
      int cc[BPL];
      double cs[BPL];
#pragma unroll
      for (int j = 0; j < BPL; ++j) { cc[j] = 0; cs[j] = 0.0; }
      auto add_pixel = [&](int pq) {
        const int* crow = cntc + pq * SS + lane;
        const double* srow = sumc + pq * SS + lane;
#pragma unroll
        for (int j = 0; j < BPL; ++j) {
          cc[j] += crow[32 * j];
          cs[j] = __dadd_rn(cs[j], srow[32 * j]);
        }
      };
      if (KHW) {
#pragma unroll
        for (int rs = 0; rs < KMAX; ++rs) add_pixel(pix0 + wofs(rs));
      } else {
        for (int rs = 0; rs < khw; ++rs) add_pixel(pix0 + win[rs]);
      }
      const int m = __shfl_sync(0xFFFFFFFFu, cc[BPL - 1], 31);
      const double T = __shfl_sync(0xFFFFFFFFu, cs[BPL - 1], 31);
      const int z = a.n - m;
      RowResult res;
      bool retry = false;
      if (m == 0) {
        res = trivial_row(false, 0.0f);  // nothing but zeros
      } else {
        // the same at the lower edge (= upper edge of the bucket before)
        int pc[BPL];
        double ps[BPL];
#pragma unroll
        for (int j = 0; j < BPL; ++j) {
          const int u = __shfl_up_sync(0xFFFFFFFFu, cc[j], 1);
          const double w = __shfl_up_sync(0xFFFFFFFFu, cs[j], 1);
          const int u0 = j ? __shfl_sync(0xFFFFFFFFu, cc[j ? j - 1 : 0], 31) : 0;
          const double w0 = j ? __shfl_sync(0xFFFFFFFFu, cs[j ? j - 1 : 0], 31) : 0.0;
          pc[j] = lane ? u : u0;
          ps[j] = lane ? w : w0;
        }
        // count and sum of the negative values (the run of zeros sits between them and the positive ones)
        int neg = 0;
        double Pneg = 0.0;
        if (qz.B0 > 0) {
          const int jn = (qz.B0 - 1) >> 5;
          int tn = 0;
          double tp = 0.0;
#pragma unroll
          for (int j = 0; j < BPL; ++j)
            if (j == jn) { tn = cc[j]; tp = cs[j]; }
          neg = __shfl_sync(0xFFFFFFFFu, tn, 31);
          Pneg = __shfl_sync(0xFFFFFFFFu, tp, 31);
        }
        // objective at the upper edge of every bucket (empty ones repeat their neighbour's split) and at the split
        // after the run of zeros; a bucket's lower edge is the upper edge of the bucket before it, except for the
        // first positive bucket, whose lower edge is the split after the zeros
        const float dz1 = (z > 0 && neg + z < a.n) ? objective_bound((double)(neg + z), Pneg, T, nd) : -1.0f;
        float best = dz1;
        float e1[BPL], bound[BPL];
#pragma unroll
        for (int j = 0; j < BPL; ++j) {
          const int b = j * 32 + lane;
          const int s1 = cc[j] + (b >= qz.B0 ? z : 0);
          e1[j] = (s1 > 0 && s1 < a.n) ? objective_bound((double)s1, cs[j], T, nd) : -1.0f;
          best = fmaxf(best, e1[j]);
        }
        float dz0 = -1.0f;  // the split before the zeros = upper edge of the last negative bucket
        if (qz.B0 > 0) {
          const int jn = (qz.B0 - 1) >> 5;
          float t = -1.0f;
#pragma unroll
          for (int j = 0; j < BPL; ++j)
            if (j == jn) t = e1[j];
          t = __shfl_sync(0xFFFFFFFFu, t, 31);
          if (z > 0) dz0 = t;
        }
#pragma unroll
        for (int j = 0; j < BPL; ++j) {
          const int b = j * 32 + lane;
          const int c = cc[j] - pc[j];
          const float up = __shfl_up_sync(0xFFFFFFFFu, e1[j], 1);
          const float wrap = j ? __shfl_sync(0xFFFFFFFFu, e1[j ? j - 1 : 0], 31) : -1.0f;
          const float d0 = (b == qz.B0 && z > 0) ? dz1 : (lane ? up : wrap);
          float dk = -1.0f;
          if (c >= 2) {
            // value bounds of the bucket and the two inner corners of the region (s, P) can visit inside it
            const int s0 = pc[j] + (b >= qz.B0 ? z : 0);
            double vlo, vhi, inv_width;
            pix_bucket_range<kOctaves>(qz, b, B, vlo, vhi, inv_width);
            const double cd = (double)c, S = cs[j] - ps[j];
            double jl = (cd * vhi - S) * inv_width;
            jl = fmin(fmax(jl, 0.0), cd);
            const double ju = cd - jl;
            dk = fmaxf(objective_bound((double)s0 + jl, ps[j] + jl * vlo, T, nd),
                       objective_bound((double)s0 + ju, ps[j] + ju * vhi, T, nd));
          }
          bound[j] = c > 0 ? fmaxf(fmaxf(d0, e1[j]), dk) : -2.0f;
        }
        best = __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, __float_as_uint(fmaxf(best, 0.0f))));
        const float need = best * prune_margin;
        int seg_lo = 1 << 20, seg_hi = -1;  // segments: buckets below B0 keep their index, the zeros are B0, the rest + 1
#pragma unroll
        for (int j = 0; j < BPL; ++j) {
          const int b = j * 32 + lane;
          if (bound[j] >= need) {
            const int seg = b + (b >= qz.B0 ? 1 : 0);
            seg_lo = min(seg_lo, seg);
            seg_hi = max(seg_hi, seg);
          }
        }
        if (z > 0 && fmaxf(dz0, dz1) >= need) { seg_lo = min(seg_lo, qz.B0); seg_hi = max(seg_hi, qz.B0); }
        seg_lo = __reduce_min_sync(0xFFFFFFFFu, seg_lo);
        seg_hi = __reduce_max_sync(0xFFFFFFFFu, seg_hi);
        const int b_lo = seg_lo > qz.B0 ? seg_lo - 1 : seg_lo;   // first bucket of the hull
        const int b_hi = seg_hi >= qz.B0 ? seg_hi - 1 : seg_hi;  // last bucket of the hull
        const int z_in = (z > 0 && seg_lo <= qz.B0 && qz.B0 <= seg_hi) ? z : 0;
        // a hull made of the zeros alone cannot be: each of their two edges is also the edge of a bucket with values
        if (!(best > 1e-30f) || seg_hi < 0 || b_lo > b_hi || b_lo < 0 || b_hi >= B) {
          retry = true;
        } else {
          int t0 = 0, t1 = 0;
          double q0 = 0.0, q1 = 0.0;
#pragma unroll
          for (int j = 0; j < BPL; ++j) {
            if (j == (b_lo >> 5)) { t0 = pc[j]; q0 = ps[j]; }
            if (j == (b_hi >> 5)) { t1 = cc[j]; q1 = cs[j]; }
          }
          const int c_below = __shfl_sync(0xFFFFFFFFu, t0, b_lo & 31);   // non-zero values below the hull
          const double P_below = __shfl_sync(0xFFFFFFFFu, q0, b_lo & 31);
          const int c_upto = __shfl_sync(0xFFFFFFFFu, t1, b_hi & 31);    // non-zero values up to its end
          const double P_upto = __shfl_sync(0xFFFFFFFFu, q1, b_hi & 31);
          const int m_sub = c_upto - c_below;
          const int s_below = c_below + (seg_lo > qz.B0 ? z : 0);  // the zeros lie below the hull
          if (m_sub < 1 || m_sub > (KHW ? kHullCapRegs : kHullCap) || (z == 0 && m_sub == a.n)) {
            retry = true;
          } else {
            // ---- gather the hull (raw bits) from the ordered lists of the window's pixels ----
            const SplitBase base{s_below, P_below, __dsub_rn(T, P_upto)};
            if (KHW) {
              // lane rs < kh*kw owns pixel rs of the window: where its part of the hull starts in its list and how
              // long it is; an exclusive scan over those lanes places the parts one after the other
              int my_pq = 0, my_st = 0, my_len = 0;
              if (lane < KMAX) {
                my_pq = pix0 + win[lane];
                const int* crow = cntc + my_pq * SS;
                my_st = b_lo > 0 ? crow[b_lo - 1] : 0;
                my_len = crow[b_hi] - my_st;
              }
              int incl = my_len;
#pragma unroll
              for (int o = 1; o < 16; o <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += t;
              }
              const int excl = incl - my_len;
              // (a one-key-per-lane search pays only where hulls of up to 32 values are the rule, i.e. under the
              // per-octave grid; elsewhere its extra code costs more in instruction fetches than it saves)
              if (__shfl_sync(0xFFFFFFFFu, incl, KMAX - 1) != m_sub) {
                retry = true;  // cannot happen; never trust a mismatch
              } else if (kOctaves && m_sub <= 32) {  // the usual case under the per-octave grid
                res = pix_gather_sort_select<1, kTable>(tile, list, C, chw, excl, my_st, my_pq, KMAX, m_sub, z_in, a.n, lane, rcp, base);
              } else if (m_sub <= 64) {
                res = pix_gather_sort_select<2, kTable>(tile, list, C, chw, excl, my_st, my_pq, KMAX, m_sub, z_in, a.n, lane, rcp, base);
              } else if (m_sub <= 128) {
                res = pix_gather_sort_select<4, kTable>(tile, list, C, chw, excl, my_st, my_pq, KMAX, m_sub, z_in, a.n, lane, rcp, base);
              } else if (m_sub <= 256) {
                res = pix_gather_sort_select<8, kTable>(tile, list, C, chw, excl, my_st, my_pq, KMAX, m_sub, z_in, a.n, lane, rcp, base);
              } else if (m_sub <= 512) {
                res = pix_gather_sort_select<16, kTable>(tile, list, C, chw, excl, my_st, my_pq, KMAX, m_sub, z_in, a.n, lane, rcp, base);
              } else {
                res = pix_gather_sort_select<32, kTable>(tile, list, C, chw, excl, my_st, my_pq, KMAX, m_sub, z_in, a.n, lane, rcp, base);
              }
            } else {
              int fill = 0;
              for (int rs = 0; rs < khw; ++rs) {
                const int pq = pix0 + win[rs];
                const int* crow = cntc + pq * SS;
                const int start = b_lo > 0 ? crow[b_lo - 1] : 0, end = crow[b_hi];
                for (int i = start + lane; i < end; i += 32)
                  scratch[fill + i - start] = __float_as_uint(tile[(int)list[pq * C + i] * chw + pq]);
                fill += end - start;
              }
              __syncwarp();
              if (fill != m_sub) retry = true;  // cannot happen; never trust a mismatch
              else if (m_sub <= 64) res = pix_sort_select<2, kTable>(scratch, m_sub, z_in, a.n, lane, rcp, base);
              else if (m_sub <= 128) res = pix_sort_select<4, kTable>(scratch, m_sub, z_in, a.n, lane, rcp, base);
              else res = pix_sort_select<8, kTable>(scratch, m_sub, z_in, a.n, lane, rcp, base);
              __syncwarp();  // the scratch array may be overwritten by the next patch
            }
            if (!retry) {
              res.K = __shfl_sync(0xFFFFFFFFu, res.K, 0);
              res.alpha = __shfl_sync(0xFFFFFFFFu, res.alpha, 0);
              res.beta = __shfl_sync(0xFFFFFFFFu, res.beta, 0);
              res.flags = 0u;
              res.tkey = __shfl_sync(0xFFFFFFFFu, res.tkey, 0);
              res.mode = __shfl_sync(0xFFFFFFFFu, res.mode, 0);
              if (res.tkey == kPadKey) retry = true;  // a split at the hull's outer edge won: not certified
            }
          }
        }
      }
      if (retry) {
        if (lane == 0 && DAB_IN_BOUNDS(pi, patch_count(a))) a.pK[pi] = kRowMark;
        continue;
      }
      if (lane == 0 && DAB_IN_BOUNDS(pi, patch_count(a))) {
        a.pK[pi] = res.K;
        a.pgamma[pi] = res.alpha;
        a.pdelta[pi] = res.beta;
        if (a.pflags) a.pflags[pi] = res.flags;
      }
      // ---- mask: bit of element (c, r, s) = [value >= threshold] (or its complement) ----
      const bool flip = res.mode == 1, none = res.mode == 2;
      const float tv = key_value(res.tkey);
      const float* origin = tile + pix0;
      if (KHW) {
        // lane = channel: its 9 bits are consecutive in the row, at bit 9*lane of the 9 words that 32 channels fill.
        // The lanes whose bits start in the same word form a run of 3 or 4 lanes: an OR over the run gives that
        // word's own bits, a second OR the bits that spill into the next word.
        const int groups = (C + 31) >> 5;
#pragma unroll 2
        for (int g = 0; g < groups; ++g) {
          const int c = g * 32 + lane;
          const bool live = c < C && !none;
          const float* src = origin + (c < C ? c : 0) * chw;
          uint32_t field = 0u;
#pragma unroll
          for (int rs = 0; rs < KMAX; ++rs) field |= ((src[wofs(rs)] >= tv) != flip) ? (1u << rs) : 0u;
          if (!live) field = 0u;
          const int sh = (lane * 9) & 31;
          uint32_t lo = field << sh, hi = sh > 23 ? field >> (32 - sh) : 0u;
          {  // OR over the run, collected in its first lane (runs are at most 4 lanes long)
            const uint32_t l1 = __shfl_down_sync(0xFFFFFFFFu, lo, 1), h1 = __shfl_down_sync(0xFFFFFFFFu, hi, 1);
            const uint32_t l2 = __shfl_down_sync(0xFFFFFFFFu, lo, 2), h2 = __shfl_down_sync(0xFFFFFFFFu, hi, 2);
            const uint32_t l3 = __shfl_down_sync(0xFFFFFFFFu, lo, 3), h3 = __shfl_down_sync(0xFFFFFFFFu, hi, 3);
            if (run_next & 1u) { lo |= l1; hi |= h1; }
            if (run_next & 2u) { lo |= l2; hi |= h2; }
            if (run_next & 4u) { lo |= l3; hi |= h3; }
          }
          // word w = own bits of run w | spill of run w - 1; lane w < 9 fetches them from the runs' first lanes
          const uint32_t own = __shfl_sync(0xFFFFFFFFu, lo, first_of_word);
          const uint32_t spill = __shfl_sync(0xFFFFFFFFu, hi, first_of_prev);
          const int w = g * 9 + lane;
          if (lane < 9 && w < a.ldp && DAB_IN_BOUNDS(pi * a.ldp + w, patch_count(a) * a.ldp))
            mrow[w] = own | (lane ? spill : 0u);
        }
        for (int w = groups * 9 + lane; w < a.ldp; w += 32)
          if (DAB_IN_BOUNDS(pi * a.ldp + w, patch_count(a) * a.ldp)) mrow[w] = 0u;
      } else {
        for (int kb = 0; kb < rounds; kb += 32) {  // 32 mask words at a time: word kb + j ends up in lane j
          const int kend = min(32, rounds - kb);
          uint32_t mine = 0;
          for (int kk = 0; kk < kend; ++kk) {
            const int i = (kb + kk) * 32 + lane;
            const bool live = i < a.n;
            const float v = origin[live ? off[i] : 0];
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, !none && live && ((v >= tv) != flip));
            if (kk == lane) mine = word;
          }
          if (lane < kend && DAB_IN_BOUNDS(pi * a.ldp + kb + lane, patch_count(a) * a.ldp)) mrow[kb + lane] = mine;
        }
        for (int w = rounds + lane; w < a.ldp; w += 32)
          if (DAB_IN_BOUNDS(pi * a.ldp + w, patch_count(a) * a.ldp)) mrow[w] = 0u;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// The kernel that follows on the stream: patches marked K = kRowMark are coded by the full sort of rowcode.cuh,
// one CTA (a group of 8 warps) per marked patch, values read straight from global memory.  Every CTA looks at a
// run of `run` (32 to 256) patch slots at a time and queues the marked ones; short runs spread the marked patches
// of a small layer over all SMs.
// ---------------------------------------------------------------------------------------------------------
template <int R>
__global__ void __launch_bounds__(kFixThreads) binarize_patches_fixup_kernel(const PixArgs a, int scratch_words, int run) {
  constexpr int W = kFixWarps;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  GroupShared* gs = reinterpret_cast<GroupShared*>(smem_raw);
  uint32_t* scratch = reinterpret_cast<uint32_t*>(gs + 1);
  int* queue = reinterpret_cast<int*>(scratch + scratch_words);
  __shared__ int qn;
  const int tig = threadIdx.x;
  const int64_t total = (int64_t)a.d.N * a.Ho * a.Wo;
  const int khw = a.d.kh * a.d.kw;
  for (int64_t chunk = (int64_t)blockIdx.x * run; chunk < total; chunk += (int64_t)gridDim.x * run) {
    __syncthreads();
    if (tig == 0) qn = 0;
    __syncthreads();
    if (tig < run && chunk + tig < total && a.pK[DAB_IDX(chunk + tig, total)] == kRowMark) queue[atomicAdd(&qn, 1)] = tig;
    __syncthreads();
    const int count = qn;
    for (int qi = 0; qi < count; ++qi) {
      const int64_t pi = chunk + queue[qi];
      const int wo = (int)(pi % a.Wo);
      const int ho = (int)((pi / a.Wo) % a.Ho);
      const int img = (int)(pi / ((int64_t)a.Wo * a.Ho));
      const float* ximg = a.x + (int64_t)img * a.d.C * a.d.H * a.d.W;
      const int hb = ho * a.d.stride_h - a.d.pad_h, wb = wo * a.d.stride_w - a.d.pad_w;
      auto keyof = [&](int i) {
        const int c = i / khw, rs = i - c * khw;
        const int r = rs / a.d.kw, s = rs - r * a.d.kw;
        const int h = hb + r, w = wb + s;
        float v = 0.0f;
        if ((unsigned)h < (unsigned)a.d.H && (unsigned)w < (unsigned)a.d.W)
          v = __ldg(ximg + DAB_IDX(((int64_t)c * a.d.H + h) * a.d.W + w, (int64_t)a.d.C * a.d.H * a.d.W));
        return order_key(v);
      };
      uint32_t kreg[R];
      group_code_row<W, R, false, false>(keyof, a.n, tig, scratch, gs, 1, nullptr, kreg);
      const RowResult res = gs->result;
      if (tig == 0 && DAB_IN_BOUNDS(pi, total)) {
        a.pK[pi] = res.K;
        a.pgamma[pi] = res.alpha;
        a.pdelta[pi] = res.beta;
        if (a.pflags) a.pflags[pi] = res.flags;
      }
      group_store_mask<W, R, false>(kreg, a.n, a.ldp, tig, res, a.pmask, pi, total);
      group_barrier(1, 32 * W);  // gs->result is overwritten by the next patch
    }
  }
}

void set_pix_tile(const dab_conv_desc& d, int Ho, int Wo, int th, int tw, PixArgs* a) {
  const int TH = th < Ho ? th : Ho, TW = tw < Wo ? tw : Wo;
  a->TH = TH; a->TW = TW;
  a->in_h = (TH - 1) * d.stride_h + d.kh;
  a->in_w = (TW - 1) * d.stride_w + d.kw;
  a->pix = a->in_h * a->in_w;
  a->ch_words = a->pix | 1;
  a->tiles_h = (Ho + TH - 1) / TH;
  a->tiles_w = (Wo + TW - 1) / TW;
}

template <int WARPS, int BPL, int KHW, typename ListT, bool kTable>
size_t pix_smem_bytes(const PixArgs& a) {
  const size_t B = 32 * BPL, SS = B + 1;
  size_t bytes = (kTable ? sizeof(double) * rcp_table_slots(a.n) : 0);
  bytes += (sizeof(double) + sizeof(int)) * (size_t)a.pix * SS;
  bytes += sizeof(float) * (size_t)a.d.C * a.ch_words;
  bytes += sizeof(uint32_t) * ((KHW ? 0 : WARPS * kHullCap) + 64) + sizeof(int) * (size_t)a.pix;
  bytes += sizeof(uint16_t) * (size_t)((a.d.kh * a.d.kw + 1) & ~1);
  if (!KHW) bytes += sizeof(uint16_t) * (size_t)((a.n + 1) & ~1);
  bytes += sizeof(ListT) * (size_t)a.pix * a.d.C;
  return (bytes + 15) & ~(size_t)15;
}

// The tile (at most 8 x 8 output positions) that fits `budget` bytes of shared memory and costs least over the whole
// layer: per tile, work in proportion to the staged values plus the rounds of patches its warps take, times the
// waves of CTAs the layer needs with `ctas_per_sm` resident.  Returns false when no shape fits.
template <int WARPS, int BPL, int KHW, typename ListT, bool kTable>
bool choose_pix_tile(PixArgs* a, size_t budget, int ctas_per_sm, size_t* smem_out, double* cost_out) {
  double best_cost = 0.0;
  int best_th = 0, best_tw = 0;
  size_t best_smem = 0;
  const double per_patch = DAB_PIX_COST_PATCH + DAB_PIX_COST_VALUE * a->n;
  const int sms = sm_count();
  for (int th = 8; th >= 1; --th) {
    for (int tw = 8; tw >= 1; --tw) {
      if ((th > a->Ho && th > 1) || (tw > a->Wo && tw > 1)) continue;
      PixArgs t = *a;
      set_pix_tile(a->d, a->Ho, a->Wo, th, tw, &t);
      if ((size_t)t.d.C * t.ch_words > 65535) continue;  // 16-bit offsets
      const size_t smem = pix_smem_bytes<WARPS, BPL, KHW, ListT, kTable>(t);
      if (smem > budget) continue;
      const int64_t tiles = (int64_t)t.tiles_h * t.tiles_w * t.d.N;
      const int64_t slots = (int64_t)sms * ctas_per_sm;
      const double waves = (double)((tiles + slots - 1) / slots);
      const int rounds = (t.TH * t.TW + WARPS - 1) / WARPS;
      const double cost = waves * (4.6 * t.pix * t.d.C + rounds * per_patch) * sqrt((double)ctas_per_sm);  // resident CTAs share the issue slots
      if (best_th == 0 || cost < best_cost) { best_cost = cost; best_th = th; best_tw = tw; best_smem = smem; }
    }
  }
  if (best_th == 0) return false;
  set_pix_tile(a->d, a->Ho, a->Wo, best_th, best_tw, a);
  *smem_out = best_smem;
  *cost_out = best_cost;
  return true;
}

constexpr size_t kSmemPerSm = 228 * 1024, kSmemCtaReserve = 1024, kSmemCtaMax = 227 * 1024;

template <int WARPS, int MINB, int BPL, int KHW, typename ListT, bool kTable>
cudaError_t launch_pix_minb(PixArgs& a, size_t smem, cudaStream_t stream) {
  auto kern = binarize_patches_pixhist_kernel<WARPS, MINB, BPL, KHW, ListT, kTable>;
  cudaError_t e = ensure_dynamic_smem(kern, smem);
  if (e != cudaSuccess) return e;
  const int64_t tiles = (int64_t)a.tiles_h * a.tiles_w * a.d.N;
  const int64_t blocks = tiles < sm_count() * MINB ? tiles : sm_count() * MINB;
  kern<<<(unsigned)blocks, WARPS * 32, smem, stream>>>(a);
  return cudaGetLastError();
}

#ifndef DAB_PIX_WIDE_FROM_BPL
#define DAB_PIX_WIDE_FROM_BPL 2   // buckets per lane from which a CTA has 16 warps instead of 8
#endif
#ifndef DAB_PIX_WARPS
#define DAB_PIX_WARPS 8
#endif
#ifndef DAB_PIX_FOUR_CTAS_UPTO_BPL
#define DAB_PIX_FOUR_CTAS_UPTO_BPL 2   // buckets per lane up to which four CTAs per SM (64 registers a thread) are tried
#endif

// Four (short rows only), three, two or one CTA per SM: the most resident CTAs whose best tile costs no more than
// 1.25 x the best of all.
template <int BPL, int KHW, typename ListT, bool kTable>
cudaError_t launch_pix(PixArgs& a, cudaStream_t stream, bool* applicable) {
  // rows of 2048 values and more leave room for one to three CTAs per SM only (tables, values and lists of a pixel
  // take 3 to 6 KB): their CTAs get twice the warps
  constexpr int W = BPL >= DAB_PIX_WIDE_FROM_BPL ? 2 * DAB_PIX_WARPS : DAB_PIX_WARPS;
  constexpr int kMostCtas = (W == DAB_PIX_WARPS && BPL <= DAB_PIX_FOUR_CTAS_UPTO_BPL) ? 4 : 3;
  PixArgs cand[4] = {a, a, a, a};
  size_t smem[4] = {0, 0, 0, 0};
  double cost[4] = {0, 0, 0, 0};
  bool ok[4] = {false, false, false, false};
  double best = 0.0;
  for (int ctas = kMostCtas; ctas >= 1; --ctas) {
    size_t budget = kSmemPerSm / ctas - kSmemCtaReserve;
    if (budget > kSmemCtaMax) budget = kSmemCtaMax;
    const int i = ctas - 1;
    ok[i] = choose_pix_tile<W, BPL, KHW, ListT, kTable>(&cand[i], budget, ctas, &smem[i], &cost[i]);
    if (ok[i] && (best == 0.0 || cost[i] < best)) best = cost[i];
  }
  *applicable = ok[0] || ok[1] || ok[2] || ok[3];
  if (!*applicable) return cudaSuccess;
  if constexpr (kMostCtas == 4) {
    if (ok[3] && cost[3] <= 1.25 * best) { a = cand[3]; return launch_pix_minb<W, 4, BPL, KHW, ListT, kTable>(a, smem[3], stream); }
  }
  if (ok[2] && cost[2] <= 1.25 * best) { a = cand[2]; return launch_pix_minb<W, 3, BPL, KHW, ListT, kTable>(a, smem[2], stream); }
  if (ok[1] && cost[1] <= 1.25 * best) { a = cand[1]; return launch_pix_minb<W, 2, BPL, KHW, ListT, kTable>(a, smem[1], stream); }
  a = cand[0];
  return launch_pix_minb<W, 1, BPL, KHW, ListT, kTable>(a, smem[0], stream);
}

// Reciprocal table for rows of fewer than 2048 values; 8-bit channel indices for up to 256 channels (3 x 3 windows;
// the general kernel, which also takes whatever falls through here, has 16-bit ones).
template <int BPL>
cudaError_t launch_pix_for(PixArgs& a, cudaStream_t stream, bool* applicable) {
  constexpr bool kTable = BPL <= 2;
  if (a.d.kh == 3 && a.d.kw == 3) {
    if (a.d.C <= 256) return launch_pix<BPL, 9, uint8_t, kTable>(a, stream, applicable);
    if constexpr (BPL >= 2) return launch_pix<BPL, 9, uint16_t, kTable>(a, stream, applicable);
  }
  return launch_pix<BPL, 0, uint16_t, kTable>(a, stream, applicable);
}

template <int R>
cudaError_t launch_fixup(const PixArgs& a, cudaStream_t stream) {
  const int sw = scratch_words_for(a.n, kFixWarps);
  const size_t smem = sizeof(GroupShared) + sizeof(uint32_t) * (size_t)sw + sizeof(int) * kFixThreads;
  auto kern = binarize_patches_fixup_kernel<R>;
  cudaError_t e = ensure_dynamic_smem(kern, smem);
  if (e != cudaSuccess) return e;
  const int64_t total = (int64_t)a.d.N * a.Ho * a.Wo;
  int run = kFixThreads;  // patch slots a CTA scans at a time: fewer for small layers, so that every SM gets some
  while (run > 32 && (total + run - 1) / run < 4 * (int64_t)sm_count()) run >>= 1;
  int64_t blocks = (total + run - 1) / run;
  if (blocks > sm_count() * 4) blocks = sm_count() * 4;
  kern<<<(unsigned)blocks, kFixThreads, smem, stream>>>(a, sw, run);
  return cudaGetLastError();
}

}  // namespace

// Patches of 257..8192 values through the pixel-histogram coder and the kernel that sorts what it marked.
// *applicable = false (nothing launched) when the geometry has no tile that fits shared memory.
cudaError_t launch_binarize_patches_pixhist(const dab_conv_desc& d, int32_t Ho, int32_t Wo, const float* x,
                                            int32_t* pK, float* pgamma, float* pdelta, uint32_t* pmask, int32_t ldp,
                                            uint32_t* pflags, cudaStream_t stream, bool* applicable) {
  PixArgs a;
  a.d = d; a.Ho = Ho; a.Wo = Wo; a.n = d.C * d.kh * d.kw;
  a.x = x; a.pK = pK; a.pgamma = pgamma; a.pdelta = pdelta; a.pflags = pflags; a.pmask = pmask; a.ldp = ldp;
  *applicable = false;
  if (a.n <= 256 || a.n > 8192 || d.kh * d.kw > 64) return cudaSuccess;
  cudaError_t e;
  // Buckets by patch length: 32 below 2048 values, 64 below 4096, 128 beyond.  Under the per-octave grids that
  // leaves a hull of about 17 values of a post-ReLU row of 576 and about 36 of a row of 1152 (with twice the buckets
  // the smaller hull saves less than tables, assembly and bounds cost; with equal-width buckets the hulls were three
  // times as long with the same number of buckets).
  if (a.n < DAB_PIX_N2) e = launch_pix_for<1>(a, stream, applicable);
  else if (a.n < DAB_PIX_N4) e = launch_pix_for<2>(a, stream, applicable);
  else e = launch_pix_for<4>(a, stream, applicable);
  if (e != cudaSuccess || !*applicable) return e;
  if (a.n <= 2048) return launch_fixup<8>(a, stream);
  if (a.n <= 4096) return launch_fixup<16>(a, stream);
  return launch_fixup<32>(a, stream);
}

}  // namespace dab

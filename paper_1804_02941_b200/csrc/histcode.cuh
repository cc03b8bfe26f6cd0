// Histogram-pruned search for the best split of one row (Section 4.1 / Algorithm 1), shared by the coder of conv
// patches and the coder of matrix rows.  One warp per row:
//   1. every non-zero value is quantised (q = floor(v * qscale)) and counted into one of B = 32*BPL buckets
//      (bucket = high bits of q): per bucket the count and the sum of the low bits of q, by shared-memory atomics;
//   2. a scan over the buckets gives, at every bucket edge, the split size s exactly and the prefix sum P to
//      within the quantisation error, hence the objective there to within a known eps; inside a bucket the
//      objective is bounded by its values at the corners of the parallelogram that the bucket's value range
//      allows (P^2/s + (T-P)^2/(n-s) is jointly convex in (s, P)).  Buckets whose bound cannot reach the best edge
//      value are discarded; the hull of the others is gathered, with exact fp64 sums of everything below and
//      above it, sorted and searched by the exact evaluator of rowcode.cuh.
// Discarding is conservative (every rounding is covered by eps), so the result is the split the full search
// finds.  The caller supplies `sweep(f)`, which calls f(value, live) once for every element of the row in any
// order (all 32 lanes together; live = false for lanes that have no element in that round).
#pragma once

#include "rowcode.cuh"

namespace dab {

// Keys the exact search takes at most (one warp sorts them, up to 32 per lane): 256 with 64 buckets (rows of fewer
// than 1024 values, where a larger scratch would cost residency), 1024 beyond.
__host__ __device__ constexpr int hist_cap(int BPL) { return BPL <= 2 ? 256 : 1024; }

// Quantisation of a row (or of a tile of rows): q = floor(v * qscale); bucket = (q >> shift) + boff.
struct Quant {
  float qscale;  // units of q per unit of value
  float u;       // value of one unit of q
  float bw;      // bucket width in units of q
  float A, R;    // largest magnitude and range of the values
  int shift, boff, B0;  // B0: first bucket of the positive values
};

// lo, hi: smallest and largest non-zero value (finite); LOG2B = log2 of the number of buckets.
__device__ __forceinline__ Quant make_quant(float lo, float hi, int qbits, int LOG2B) {
  Quant qz;
  const int B = 1 << LOG2B;
  qz.shift = qbits - LOG2B;
  if (lo >= 0.0f) {         // no negative value: q in [0, 2^qbits)
    qz.qscale = __fdividef((float)(1 << qbits) * 0.99999f, fmaxf(hi, 1e-37f));
    qz.boff = 0; qz.B0 = 0;
  } else if (hi <= 0.0f) {  // no positive value: q in [-2^qbits, 0)
    qz.qscale = __fdividef((float)(1 << qbits) * 0.99999f, -lo);
    qz.boff = B; qz.B0 = B;
  } else {                  // both signs: q in [-2^(qbits-1), 2^(qbits-1))
    qz.qscale = __fdividef((float)(1 << (qbits - 1)) * 0.99999f, fmaxf(-lo, hi));
    qz.boff = B / 2; qz.B0 = B / 2;
  }
  qz.u = __fdividef(1.0f, qz.qscale);
  qz.bw = (float)(1 << qz.shift);
  qz.A = fmaxf(fabsf(lo), fabsf(hi));
  qz.R = hi - lo;
  return qz;
}

// Bits of q: 24 (fp32 holds them), fewer if the sum of n in-bucket offsets (qbits - LOG2B bits each) could leave 32 bits.
__host__ __device__ inline int quant_bits(int n, int LOG2B) {
  int qbits = 24;
  while (((long long)n << (qbits - LOG2B)) >= 0x7FFFFFFFll) --qbits;
  return qbits;
}

__device__ __forceinline__ float objective_f32(float s, float P, float T, float n) {
  // P^2/s + (T-P)^2/(n-s) with the limits 0 at s = 0 (P = 0 there) and s = n
  const float Q = T - P;
  const float a = s > 0.0f ? __fdividef(P * P, s) : 0.0f;
  const float b = n - s > 0.0f ? __fdividef(Q * Q, n - s) : 0.0f;
  return a + b;
}

template <int E>
__device__ __noinline__ RowResult hist_sort_select(const uint32_t* scratch, int m, int z, int n, int lane,
                                                   const double* rcp, const SplitBase base) {
  uint32_t r[E];
#pragma unroll
  for (int j = 0; j < E; ++j) {
    const int idx = j * 32 + lane;
    r[j] = idx < m ? order_key(__uint_as_float(scratch[idx])) : kPadKey;   // the gather stored raw bits
  }
  group_sort<1, E>(r, lane, nullptr, 0);
  return group_select<1, E, true, true>(r, m, z, n, lane, nullptr, 0, rcp, base);
}

// The search.  hist: B (count, sum) pairs and scratch: hist_cap(BPL) words of shared memory owned by the warp; rcp: the
// table of n + 1 reciprocals.  Returns false when the row is left to the sorting coder (a hull of more than
// hist_cap(BPL) values, or a winner at the hull's outer edge); otherwise res holds the code (in every lane).
template <int BPL, typename Sweep>
__device__ __forceinline__ bool hist_search(Sweep sweep, int n, const Quant& qz, int2* hist, uint32_t* scratch,
                                            const double* rcp, int lane, RowResult& res) {
  constexpr int B = 32 * BPL;
  constexpr int kHistCap = hist_cap(BPL);
  const int qmask = (1 << qz.shift) - 1;
  const float nf = (float)n;
  const unsigned lt = (1u << lane) - 1u;
  // ---- pass 1: histogram (the order of the elements does not matter: lane = channel, loop over the window) ----
#pragma unroll
  for (int j = 0; j < BPL; ++j) hist[lane * BPL + j] = make_int2(0, 0);
  __syncwarp();
  sweep([&](float v, bool live) {
    const int q = __float2int_rd(v * qz.qscale);
    const int b = min(max((q >> qz.shift) + qz.boff, 0), B - 1);
    if (live && v != 0.0f) {
      atomicAdd(&hist[b].x, 1);
      atomicAdd(&hist[b].y, q & qmask);
    }
  });
  __syncwarp();
  // ---- scan over the buckets: lane owns buckets lane*BPL .. lane*BPL+BPL-1 ----
  int c[BPL];
  double Q[BPL];   // sum of q over the bucket: count * first q of the bucket + sum of the offsets (exact)
  int csum = 0;
  double qsum = 0.0;
#pragma unroll
  for (int j = 0; j < BPL; ++j) {
    const int2 hq = hist[lane * BPL + j];
    c[j] = hq.x;
    Q[j] = (double)hq.x * (double)((lane * BPL + j - qz.boff) * (1 << qz.shift)) + (double)(unsigned)hq.y;
    csum += hq.x; qsum += Q[j];
  }
  int cincl = csum;
  double qincl = qsum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int co = __shfl_up_sync(0xFFFFFFFFu, cincl, o);
    const double qo = __shfl_up_sync(0xFFFFFFFFu, qincl, o);
    if (lane >= o) { cincl += co; qincl += qo; }
  }
  const int m = __shfl_sync(0xFFFFFFFFu, cincl, 31);
  const double QT = __shfl_sync(0xFFFFFFFFu, qincl, 31);
  const int z = n - m;
  bool retry = false;
  if (m == 0) {
    res = trivial_row(false, 0.0f);  // nothing but zeros
  } else {
    // nominal prefix sums in units of qz.u: every value lies in [(q - 1) qz.u, (q + 2) qz.u], centre (q + 0.5) qz.u
    const float Tn = ((float)QT + 0.5f * (float)m) * qz.u;
    const float eps_fixed = 3.0f * (qz.R + qz.A) * (float)m * qz.u;          // effect of the quantisation on any objective value
    int cbefore = cincl - csum;
    double qbefore = qincl - qsum;
    float best_edge = -1.0f;
    float bound[BPL];
    int negc_local = 0;
#pragma unroll
    for (int j = 0; j < BPL; ++j) {
      const int b = lane * BPL + j;
      const float s0 = (float)(cbefore + (b >= qz.B0 ? z : 0));
      const float P0 = ((float)qbefore + 0.5f * (float)cbefore) * qz.u;
      const int cafter = cbefore + c[j];
      const double qafter = qbefore + Q[j];
      const float s1 = s0 + (float)c[j];
      const float P1 = ((float)qafter + 0.5f * (float)cafter) * qz.u;
      float d0 = -1.0f, d1 = -1.0f, dk = -1.0f;
      if (s0 > 0.0f && s0 < nf) d0 = objective_f32(s0, P0, Tn, nf);
      if (s1 > 0.0f && s1 < nf) d1 = objective_f32(s1, P1, Tn, nf);
      best_edge = fmaxf(best_edge, fmaxf(d0, d1));
      if (c[j] >= 2) {
        // value range of the bucket, and the two inner corners of the region (s, P) can visit inside it
        const float qlo = (float)(b - qz.boff) * qz.bw;
        const float va = (qlo - 1.0f) * qz.u, vb = (qlo + qz.bw + 2.0f) * qz.u;
        const float cf = (float)c[j], sig = P1 - P0;
        float jl = __fdividef(cf * vb - sig, vb - va);
        jl = fminf(fmaxf(jl, 0.0f), cf);
        const float ju = cf - jl;
        dk = fmaxf(objective_f32(s0 + jl, P0 + jl * va, Tn, nf), objective_f32(s0 + ju, P0 + ju * vb, Tn, nf));
        // the corners move with the uncertainty of the bucket's sum: 1.5 c qz.u in P, that over (vb - va) in s
        dk += (qz.A * qz.A + 2.0f * qz.R * qz.A) * __fdividef(1.5f * cf * qz.u, vb - va) + 2.0f * qz.R * 1.5f * cf * qz.u;
      }
      bound[j] = c[j] > 0 ? fmaxf(fmaxf(d0, d1), dk) : -2.0f;
      if (b < qz.B0) negc_local += c[j];
      cbefore = cafter; qbefore = qafter;
    }
    const int negc = __reduce_add_sync(0xFFFFFFFFu, negc_local);
    // the two splits around the run of zeros (their sums are those of the negatives)
    const double qneg = __shfl_sync(0xFFFFFFFFu, qincl, max(qz.B0 / BPL - 1, 0));   // inclusive sum up to bucket qz.B0-1
    const float Pneg = qz.B0 > 0 ? ((float)qneg + 0.5f * (float)negc) * qz.u : 0.0f;
    float dz0 = -1.0f, dz1 = -1.0f;
    if (z > 0) {
      if (negc > 0) dz0 = objective_f32((float)negc, Pneg, Tn, nf);
      if (negc + z < n) dz1 = objective_f32((float)(negc + z), Pneg, Tn, nf);
    }
    best_edge = fmaxf(best_edge, fmaxf(dz0, dz1));
    best_edge = __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, __float_as_uint(fmaxf(best_edge, 0.0f))));
    // a bucket (or the zero run) survives if its bound, raised by every rounding, reaches the best edge lowered by them
    const float slack = 2.0f * eps_fixed + 2e-4f * best_edge;
    const float need = best_edge - slack;
    int seg_lo = 1 << 20, seg_hi = -1;
#pragma unroll
    for (int j = 0; j < BPL; ++j) {
      const int b = lane * BPL + j;
      if (c[j] > 0 && bound[j] + slack >= need) {
        const int seg = b + (b >= qz.B0 ? 1 : 0);
        seg_lo = min(seg_lo, seg);
        seg_hi = max(seg_hi, seg);
      }
    }
    if (z > 0 && fmaxf(dz0, dz1) + slack >= need) { seg_lo = min(seg_lo, qz.B0); seg_hi = max(seg_hi, qz.B0); }
    seg_lo = __reduce_min_sync(0xFFFFFFFFu, seg_lo);
    seg_hi = __reduce_max_sync(0xFFFFFFFFu, seg_hi);
    // hull in bucket and q terms
    const int b_lo = seg_lo > qz.B0 ? seg_lo - 1 : seg_lo;          // first bucket of the hull (seg_lo == qz.B0: bucket qz.B0)
    const int b_hi = seg_hi >= qz.B0 ? seg_hi - 1 : seg_hi;         // last bucket of the hull (seg_hi == qz.B0: bucket qz.B0-1)
    const int z_in = (z > 0 && seg_lo <= qz.B0 && qz.B0 <= seg_hi) ? z : 0;
    int msub_local = 0, sbelow_local = 0;
#pragma unroll
    for (int j = 0; j < BPL; ++j) {
      const int b = lane * BPL + j;
      if (b >= b_lo && b <= b_hi) msub_local += c[j];
      if (b < b_lo) sbelow_local += c[j];
    }
    const int m_sub = __reduce_add_sync(0xFFFFFFFFu, msub_local);
    int s_below = __reduce_add_sync(0xFFFFFFFFu, sbelow_local);
    if (seg_lo > qz.B0) s_below += z;                               // the zeros lie below the hull
    // (a constant row has all its values in one bucket: with more than kHistCap values it is left to the group kernel)
    if (seg_hi < 0 || m_sub < 1 || m_sub > kHistCap || (z == 0 && m_sub == n)) {
      retry = true;
    } else {
      const int qA = (b_lo - qz.boff) * (1 << qz.shift);               // q range of the hull's buckets
      const int qB = (b_hi + 1 - qz.boff) * (1 << qz.shift) - 1;
      const bool open_lo = b_lo == 0, open_hi = b_hi == B - 1;   // the end buckets take whatever falls outside the range
      // ---- pass 2: gather the hull (raw bits), exact sums of what lies below and above it ----
      double below = 0.0, above = 0.0;
      int cnt = 0;
      sweep([&](float v, bool live) {
        const int q = __float2int_rd(v * qz.qscale);
        const bool nz = live && v != 0.0f;
        const bool lowq = nz && q < qA && !open_lo, highq = nz && q > qB && !open_hi;
        const bool in = nz && !lowq && !highq;
        const double dv = (double)v;
        below = __dadd_rn(below, lowq ? dv : 0.0);
        above = __dadd_rn(above, highq ? dv : 0.0);
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, in);
        if (in) scratch[min(cnt + __popc(bal & lt), kHistCap - 1)] = __float_as_uint(v);
        cnt += __popc(bal);
      });
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        below = __dadd_rn(below, __shfl_xor_sync(0xFFFFFFFFu, below, o));
        above = __dadd_rn(above, __shfl_xor_sync(0xFFFFFFFFu, above, o));
      }
      __syncwarp();
      if (cnt != m_sub) {
        retry = true;                                            // cannot happen; never trust a mismatch
      } else {
        const SplitBase base{s_below, below, above};
        if (m_sub <= 64) res = hist_sort_select<2>(scratch, m_sub, z_in, n, lane, rcp, base);
        else if (m_sub <= 128) res = hist_sort_select<4>(scratch, m_sub, z_in, n, lane, rcp, base);
        else if (m_sub <= 256) res = hist_sort_select<8>(scratch, m_sub, z_in, n, lane, rcp, base);
        else if (kHistCap > 256 && m_sub <= 512) res = hist_sort_select<16>(scratch, m_sub, z_in, n, lane, rcp, base);
        else if (kHistCap > 256) res = hist_sort_select<32>(scratch, m_sub, z_in, n, lane, rcp, base);
        res.K = __shfl_sync(0xFFFFFFFFu, res.K, 0);
        res.alpha = __shfl_sync(0xFFFFFFFFu, res.alpha, 0);
        res.beta = __shfl_sync(0xFFFFFFFFu, res.beta, 0);
        res.flags = 0u;
        res.tkey = __shfl_sync(0xFFFFFFFFu, res.tkey, 0);
        res.mode = __shfl_sync(0xFFFFFFFFu, res.mode, 0);
        if (res.tkey == kPadKey) retry = true;                   // a split at the hull's outer edge won: not certified
      }
      __syncwarp();
    }
  }
  return !retry;
}

}  // namespace dab

// Core of the row coder: a group of W warps turns one row of n fp32 values (read through an accessor)
// into K, alpha, beta and the packed mask.
//
// Steps, all inside the group:
//   1. compaction  - keys of the non-zero values go to a scratch array; exact zeros are only counted.
//                    Equal values never straddle the best split, so the whole run of zeros is handled
//                    as one block of z elements with sum 0 at its place in the sorted order.
//   2. sort        - bitonic network on registers, E keys per thread, blocked layout (thread t owns
//                    sorted positions t*E .. t*E+E-1): strides below E stay inside a thread, strides
//                    below 32E use warp shuffles, larger ones go through shared memory.  Every merge
//                    starts with a mirror stage so that all compare-exchanges sort upwards.
//   3. scan        - fp64 running sums of the sorted values (thread-local, then across the group).
//   4. objective   - D_s of Algorithm 1 at every split between distinct values.  A first pass uses
//                    a table of correctly rounded reciprocals instead of divisions (error < 1e-15
//                    relative) to find the maximum; a second pass evaluates the exactly rounded
//                    expression only for splits within 1e-13 of that maximum and takes the arg-max of
//                    (D, s) with "largest s wins ties".
//   5. outputs     - orientation by |mean|, alpha/beta rounded once to fp32, threshold key for the mask.
#pragma once

#include "common.cuh"

namespace dab {

constexpr int kWarpsPerCta = 8;             // warps of a CTA in the one-warp-per-row kernels
constexpr uint32_t kZeroKey = 0x80000000u;  // order_key(0.0f)

// Scratch words a group of W warps needs for rows of up to n values (the largest sort capacity reachable).
inline int scratch_words_for(int n, int W) {
  int cap = 128 * W;
  while (cap < n) cap <<= 1;
  return cap;
}
constexpr double kBand = 1.0 - 1e-13;       // splits whose approximate objective is below max*kBand cannot win

__device__ __forceinline__ void group_barrier(int bar_id, int threads) {
  if (threads == 32)
    __syncwarp();
  else
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(threads) : "memory");
}

// Ascending bitonic sort of 32*W*E keys, E per thread, blocked layout.
template <int W, int E>
__device__ __forceinline__ void group_sort(uint32_t (&r)[E], int tig, uint32_t* xbuf, int bar_id) {
  constexpr int NTOT = 32 * W * E;
  constexpr int GT = 32 * W;
  const int ibase = tig * E;
#pragma unroll
  for (int k = 2; k <= NTOT; k <<= 1) {
    // mirror stage: element i meets element i ^ (k-1); the lower index keeps the minimum
    if (k <= E) {
#pragma unroll
      for (int j = 0; j < E; ++j) {
        const int p = j ^ (k - 1);
        if (j < p) {
          uint32_t lo = min(r[j], r[p]), hi = max(r[j], r[p]);
          r[j] = lo;
          r[p] = hi;
        }
      }
    } else {
      const int tx = k / E - 1;  // partner thread = tig ^ tx, partner register = E-1-j
      const bool lower = (ibase & (k >> 1)) == 0;
      if (tx >= 32) {
#pragma unroll
        for (int j = 0; j < E; ++j) xbuf[j * GT + tig] = r[j];
        group_barrier(bar_id, GT);
#pragma unroll
        for (int j = 0; j < E; ++j) {
          uint32_t o = xbuf[(E - 1 - j) * GT + (tig ^ tx)];
          r[j] = lower ? min(r[j], o) : max(r[j], o);
        }
        group_barrier(bar_id, GT);
      } else {
        uint32_t o[E];
#pragma unroll
        for (int j = 0; j < E; ++j) o[j] = __shfl_xor_sync(0xFFFFFFFFu, r[E - 1 - j], tx);
#pragma unroll
        for (int j = 0; j < E; ++j) r[j] = lower ? min(r[j], o[j]) : max(r[j], o[j]);
      }
    }
    // half-cleaners: element i meets i ^ st
#pragma unroll
    for (int st = k >> 2; st >= 1; st >>= 1) {
      if (st >= 32 * E) {
        const bool lower = (ibase & st) == 0;
#pragma unroll
        for (int j = 0; j < E; ++j) xbuf[j * GT + tig] = r[j];
        group_barrier(bar_id, GT);
#pragma unroll
        for (int j = 0; j < E; ++j) {
          uint32_t o = xbuf[j * GT + (tig ^ (st / E))];
          r[j] = lower ? min(r[j], o) : max(r[j], o);
        }
        group_barrier(bar_id, GT);
      } else if (st >= E) {
        const bool lower = (ibase & st) == 0;
#pragma unroll
        for (int j = 0; j < E; ++j) {
          uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, r[j], st / E);
          r[j] = lower ? min(r[j], o) : max(r[j], o);
        }
      } else {
#pragma unroll
        for (int j = 0; j < E; ++j) {
          if ((j & st) == 0) {
            uint32_t lo = min(r[j], r[j | st]), hi = max(r[j], r[j | st]);
            r[j] = lo;
            r[j | st] = hi;
          }
        }
      }
    }
  }
}

struct RowResult {
  int K;
  float alpha, beta;
  uint32_t flags;
  uint32_t tkey;  // mask bit i = (key_i >= tkey) != (mode == 1)
  int mode;       // 0: e = [w >= t], 1: e = [w < t], 2: empty mask
};

struct GroupShared {   // per group of more than one warp, in shared memory
  double wsum[32];     // per-warp sums
  double wmax[32];     // per-warp maxima of the approximate objective
  int wneg[32];        // per-warp counts of negative keys
  uint32_t wfirst[33]; // first key of each warp (index W: pad key)
  long long wbestD[32];
  int wbestS[32];
  double wbestP[32];
  uint32_t wbestT[32];
  int wcnt[32];        // per-warp counts of non-zero keys
  uint32_t wkmin[32];  // per-warp smallest and largest key
  uint32_t wkmax[32];
  RowResult result;
};

// Table of correctly rounded reciprocals 1/s, s = 1..n.  Lanes of a warp look up values of s that are E apart
// (E = 4, 8, 16, 32), so entry s lives at slot s + s/16: one pad slot per 16 entries spreads such accesses over
// the banks of shared memory.
__device__ __forceinline__ int rcp_slot(int s) { return s + (s >> 4); }
__host__ __device__ inline int rcp_table_slots(int n) { return n + (n >> 4) + 2; }

__device__ __forceinline__ void fill_reciprocals(double* rcp, int n, int tid, int threads) {
  for (int s = tid; s <= n; s += threads) rcp[rcp_slot(s)] = s ? __drcp_rn((double)s) : 0.0;
}

// Objective with reciprocals from the table: within 1e-15 relative of the exactly rounded expression, both
// terms being non-negative.
__device__ __forceinline__ double objective_fast(double P, double T, int s, int n, const double* rcp) {
  double Q = T - P;
  return fma(Q * Q, rcp[rcp_slot(n - s)], (P * P) * rcp[rcp_slot(s)]);
}

__device__ __forceinline__ RowResult finish_row(double bP, int bS, uint32_t bT, double T, int n) {
  double m_lo = __ddiv_rn(bP, (double)bS);
  double m_hi = __ddiv_rn(__dsub_rn(T, bP), (double)(n - bS));
  bool low_side = fabs(m_lo) > fabs(m_hi);  // e marks the partition whose mean is larger in magnitude
  RowResult res;
  res.K = low_side ? bS : n - bS;
  res.alpha = (float)(low_side ? m_lo : m_hi);
  res.beta = (float)(low_side ? m_hi : m_lo);
  res.flags = 0u;
  res.tkey = bT;
  res.mode = low_side ? 1 : 0;
  return res;
}

__device__ __forceinline__ RowResult trivial_row(bool bad, float value) {
  RowResult res;
  res.K = 0;
  float c = bad ? __uint_as_float(0x7FC00000u) : value;
  res.alpha = c;
  res.beta = c;
  res.flags = bad ? DAB_ROW_NONFINITE : DAB_ROW_DEGENERATE;
  res.tkey = 0u;
  res.mode = 2;
  return res;
}

// Objective evaluation over the sorted keys in r[] (blocked layout: this thread owns sorted non-zero positions
// q0 .. q0+E-1 of m), z zeros elsewhere in the row, n row length.  The result is valid in thread 0 of the group.
//
// kTable (rcp = table of n+1 reciprocals): every admissible split gets the fast objective; the splits within
// 1e-13 of the maximum are the contenders.  One contender (the usual case) wins outright; several are
// re-evaluated with the exactly rounded expression and compared as (D, s).  Without the table every split is
// evaluated exactly.
//
// SplitBase: the keys in r[] may be a contiguous run of the row's sorted order instead of all of it; then s_below
// elements with sum P_below precede them and elements with sum P_above follow (m, z, and the zero run refer to
// the run; n to the whole row).  The split before the first key of the run is not evaluated.
struct SplitBase {
  int s_below;
  double P_below, P_above;
};

template <int W, int E, bool kTable, bool kBased = false>
__device__ __forceinline__ RowResult group_select(const uint32_t (&r)[E], int m, int z, int n, int tig,
                                                  GroupShared* gs, int bar_id, const double* rcp,
                                                  const SplitBase base = SplitBase{0, 0.0, 0.0}) {
  const int sb = kBased ? base.s_below : 0;
  constexpr int GT = 32 * W;
  constexpr bool kKeep = kTable && (E <= 8);  // keep fp64 values and fast objectives of this thread in registers
  const int lane = tig & 31, warp = tig >> 5;
  const int q0 = tig * E;

  double loc[kKeep ? E : 1];  // loc[j] = sum of this thread's sorted values 0..j
  double local = 0.0;
  int negc = 0;
#pragma unroll
  for (int j = 0; j < E; ++j) {
    const bool in = q0 + j < m;
    double vj = in ? (double)key_value(r[j]) : 0.0;
    local = __dadd_rn(local, vj);
    if (kKeep) loc[kKeep ? j : 0] = local;
    negc += in && (r[j] < kZeroKey);
  }
  double incl = local;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    double o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
    if (lane >= off) incl = __dadd_rn(incl, o);
  }
  int neg = __reduce_add_sync(0xFFFFFFFFu, negc);
  uint32_t next_first = __shfl_down_sync(0xFFFFFFFFu, r[0], 1);  // first key of the next thread
  double before = 0.0, T;
  if (W > 1) {
    if (lane == 31) gs->wsum[warp] = incl;
    if (lane == 0) {
      gs->wneg[warp] = neg;
      gs->wfirst[warp] = r[0];
      if (warp == 0) gs->wfirst[W] = kPadKey;
    }
    group_barrier(bar_id, GT);
    T = 0.0;
    neg = 0;
#pragma unroll
    for (int w = 0; w < W; ++w) {
      double ws = gs->wsum[w];
      if (w < warp) before = __dadd_rn(before, ws);
      T = __dadd_rn(T, ws);
      neg += gs->wneg[w];
    }
    if (lane == 31) next_first = gs->wfirst[warp + 1];
  } else {
    T = __shfl_sync(0xFFFFFFFFu, incl, 31);
    if (lane == 31) next_first = kPadKey;
  }
  if (kBased) {
    T = __dadd_rn(__dadd_rn(base.P_below, T), base.P_above);
    before = __dadd_rn(before, base.P_below);
  }
  double excl = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
  if (lane == 0) excl = 0.0;
  const double P0 = __dadd_rn(before, excl);  // sum of everything sorted before this thread's keys

  // Split "after sorted non-zero q": s = q+1 (q negative) or q+1+z; admissible iff q < m, s < n and the next key
  // differs (the pad key behind the last real key always differs).  Split "after the zeros": s = neg+z, owned
  // by the thread that holds q == neg, admissible iff z > 0 and neg < m.
  const bool owns_zero_split = (z > 0) && (neg < m) && (neg >= q0) && (neg < q0 + E);

  double bD = -1.0, bP = 0.0;
  int bS = 0;
  uint32_t bT = 0;
  bool several = true;

  if (kKeep) {
    double Dj[kKeep ? E : 1];
    // prefix sum up to and including sorted position q0+j: P0 + loc[j] (the same expression wherever it is needed)
    double lmax = 0.0, Pz = P0;
#pragma unroll
    for (int j = 0; j < E; ++j) {
      const int q = q0 + j;
      const double P = __dadd_rn(P0, loc[kKeep ? j : 0]);
      if (q + 1 == neg) Pz = P;  // sum of the negatives (P0 itself when neg == q0)
      const int s = sb + q + 1 + (q >= neg ? z : 0);
      const uint32_t kn = (j + 1 < E) ? r[(j + 1 < E) ? j + 1 : j] : next_first;
      const bool ok = (q < m) && (s < n) && (r[j] != kn);
      double D = ok ? objective_fast(P, T, s, n, rcp) : -1.0;
      Dj[kKeep ? j : 0] = D;
      lmax = fmax(lmax, D);
    }
    const double Dz = owns_zero_split ? objective_fast(Pz, T, sb + neg + z, n, rcp) : -1.0;
    lmax = fmax(lmax, Dz);
    // maximum over the group (lmax >= 0: its bit pattern orders like an integer)
    long long b = __double_as_longlong(lmax);
    int hi = (int)(b >> 32);
    int hmax = __reduce_max_sync(0xFFFFFFFFu, hi);
    unsigned lo = (hi == hmax) ? (unsigned)b : 0u;
    unsigned lmx = __reduce_max_sync(0xFFFFFFFFu, lo);
    double gmax = __longlong_as_double(((long long)hmax << 32) | (long long)lmx);
    if (W > 1) {
      if (lane == 0) gs->wmax[warp] = gmax;
      group_barrier(bar_id, GT);
#pragma unroll
      for (int w = 0; w < W; ++w) gmax = fmax(gmax, gs->wmax[w]);
    }
    const double thr = gmax * kBand;
    unsigned cmask = (Dz >= thr) ? (1u << (E & 31)) : 0u;  // this branch exists for E <= 8 only
#pragma unroll
    for (int j = 0; j < E; ++j) cmask |= (Dj[kKeep ? j : 0] >= thr) ? (1u << j) : 0u;
    int total = __reduce_add_sync(0xFFFFFFFFu, __popc(cmask));
    if (W > 1) {
      if (lane == 0) gs->wneg[warp] = total;  // wneg is free again
      group_barrier(bar_id, GT);
      total = 0;
#pragma unroll
      for (int w = 0; w < W; ++w) total += gs->wneg[w];
    }
    several = total > 1;
    while (cmask) {
      const int j = __ffs(cmask) - 1;
      cmask &= cmask - 1;
      double Pc;
      int s;
      uint32_t tk;
      if (j == E) {
        Pc = Pz;
        s = sb + neg + z;
        tk = kPadKey;
#pragma unroll
        for (int i = 0; i < E; ++i)
          if (q0 + i == neg) tk = r[i];  // first key above the zeros
      } else {
        double lj = 0.0;
        tk = next_first;
#pragma unroll
        for (int i = 0; i < E; ++i) {
          if (i == j) lj = loc[kKeep ? i : 0];
          if (i == j + 1) tk = r[i];
        }
        Pc = __dadd_rn(P0, lj);
        const int q = q0 + j;
        s = sb + q + 1 + (q >= neg ? z : 0);
        if (q == neg - 1 && z > 0) tk = kZeroKey;  // the zeros are the smallest values of the high side
      }
      const double D = several ? objective(Pc, T, s, n) : 1.0;
      if (D > bD || (D == bD && s > bS)) { bD = D; bP = Pc; bS = s; bT = tk; }
    }
  } else {
    double thr = -1.0;
    if (kTable) {  // pass 1: maximum of the fast objective
      double P = P0, lmax = 0.0;
#pragma unroll
      for (int j = 0; j < E; ++j) {
        const int q = q0 + j;
        if (q < m) {
          const uint32_t kc = r[j];
          const uint32_t kn = (j + 1 < E) ? r[(j + 1 < E) ? j + 1 : j] : next_first;
          if (q == neg && owns_zero_split) lmax = fmax(lmax, objective_fast(P, T, sb + neg + z, n, rcp));
          P = __dadd_rn(P, (double)key_value(kc));
          const int s = sb + q + 1 + (q >= neg ? z : 0);
          if (s < n && kc != kn) lmax = fmax(lmax, objective_fast(P, T, s, n, rcp));
        }
      }
      long long b = __double_as_longlong(lmax);
      int hi = (int)(b >> 32);
      int hmax = __reduce_max_sync(0xFFFFFFFFu, hi);
      unsigned lo = (hi == hmax) ? (unsigned)b : 0u;
      unsigned lmx = __reduce_max_sync(0xFFFFFFFFu, lo);
      double gmax = __longlong_as_double(((long long)hmax << 32) | (long long)lmx);
      if (W > 1) {
        if (lane == 0) gs->wmax[warp] = gmax;
        group_barrier(bar_id, GT);
#pragma unroll
        for (int w = 0; w < W; ++w) gmax = fmax(gmax, gs->wmax[w]);
      }
      thr = gmax * kBand;
    }
    // pass 2: exactly rounded objective (of the contenders only, when the table is in use)
    double P = P0;
#pragma unroll
    for (int j = 0; j < E; ++j) {
      const int q = q0 + j;
      if (q < m) {
        const uint32_t kc = r[j];
        const uint32_t kn = (j + 1 < E) ? r[(j + 1 < E) ? j + 1 : j] : next_first;
        if (q == neg && owns_zero_split) {
          const int s = sb + neg + z;
          if (!kTable || objective_fast(P, T, s, n, rcp) >= thr) {
            double D = objective(P, T, s, n);
            if (D >= bD) { bD = D; bP = P; bS = s; bT = kc; }
          }
        }
        P = __dadd_rn(P, (double)key_value(kc));
        const int s = sb + q + 1 + (q >= neg ? z : 0);
        if (s < n && kc != kn) {
          if (!kTable || objective_fast(P, T, s, n, rcp) >= thr) {
            double D = objective(P, T, s, n);
            if (D >= bD) {  // ascending s: ">=" keeps the largest s among equal objectives
              bD = D; bP = P; bS = s;
              bT = (q == neg - 1 && z > 0) ? kZeroKey : kn;
            }
          }
        }
      }
    }
  }

  int src;
  if (!several) {  // a single contender in the whole group: no comparison needed
    const unsigned own = __ballot_sync(0xFFFFFFFFu, bD > 0.0);
    src = own ? __ffs(own) - 1 : 0;
  } else {
    // arg-max of (D, s): D >= 0 (or -1 for "none"), so its bits order like a signed 64-bit integer
    long long dbits = __double_as_longlong(bD);
    int hi = (int)(dbits >> 32);
    int hmax = __reduce_max_sync(0xFFFFFFFFu, hi);
    unsigned lo = (hi == hmax) ? (unsigned)dbits : 0u;
    unsigned lmax2 = __reduce_max_sync(0xFFFFFFFFu, lo);
    bool top = (hi == hmax) && ((unsigned)dbits == lmax2);
    int smax = __reduce_max_sync(0xFFFFFFFFu, top ? bS : -1);
    src = __ffs(__ballot_sync(0xFFFFFFFFu, top && bS == smax)) - 1;
  }
  bD = __shfl_sync(0xFFFFFFFFu, bD, src);
  bP = __shfl_sync(0xFFFFFFFFu, bP, src);
  bT = __shfl_sync(0xFFFFFFFFu, bT, src);
  bS = __shfl_sync(0xFFFFFFFFu, bS, src);
  if (W > 1) {
    if (lane == 0) {
      gs->wbestD[warp] = __double_as_longlong(bD);
      gs->wbestS[warp] = bS;
      gs->wbestP[warp] = bP;
      gs->wbestT[warp] = bT;
    }
    group_barrier(bar_id, GT);
    if (tig == 0) {
      long long best = gs->wbestD[0];
      int bw = 0;
      for (int w = 1; w < W; ++w) {
        long long d = gs->wbestD[w];
        if (d > best || (d == best && gs->wbestS[w] > gs->wbestS[bw])) { best = d; bw = w; }
      }
      bS = gs->wbestS[bw];
      bP = gs->wbestP[bw];
      bT = gs->wbestT[bw];
    }
  }
  RowResult res;
  if (W == 1) {
    // every lane holds the winner: the two means are formed side by side in lanes 0 and 1 (the same two divisions as
    // finish_row, one after the other's latency instead of behind it)
    const double num = lane == 1 ? __dsub_rn(T, bP) : bP;
    const double den = lane == 1 ? (double)(n - bS) : (double)bS;
    const double mean = __ddiv_rn(num, den);
    const double m_lo = __shfl_sync(0xFFFFFFFFu, mean, 0), m_hi = __shfl_sync(0xFFFFFFFFu, mean, 1);
    const bool low_side = fabs(m_lo) > fabs(m_hi);
    res.K = low_side ? bS : n - bS;
    res.alpha = (float)(low_side ? m_lo : m_hi);
    res.beta = (float)(low_side ? m_hi : m_lo);
    res.flags = 0u;
    res.tkey = bT;
    res.mode = low_side ? 1 : 0;
    return res;
  }
  if (tig == 0) res = finish_row(bP, bS, bT, T, n);
  return res;
}

// ---------------------------------------------------------------------------------------------------------
// Groups of several warps (rows longer than 1024 values)
// ---------------------------------------------------------------------------------------------------------
template <int W, int E, bool kTable>
__device__ __noinline__ void group_sort_select(uint32_t* scratch, int m, int z, int n, int tig, GroupShared* gs,
                                               int bar_id, const double* rcp) {
  constexpr int GT = 32 * W;
  uint32_t r[E];
#pragma unroll
  for (int j = 0; j < E; ++j) {  // the keys are unsorted: any assignment of keys to positions will do
    int idx = j * GT + tig;
    r[j] = idx < m ? scratch[idx] : kPadKey;
  }
  group_barrier(bar_id, GT);  // scratch is reused for the cross-warp exchanges
  group_sort<W, E>(r, tig, scratch, bar_id);
  RowResult res = group_select<W, E, kTable>(r, m, z, n, tig, gs, bar_id, rcp);
  if (tig == 0) gs->result = res;
}

// Codes one row with a group of W > 1 warps.  `keyof(i)` returns the order-preserving key of element i (0 <= i < n).  Warp w of the group
// owns rounds w*R .. w*R+R-1 of the row (element (round)*32 + lane) and keeps their keys in kreg[], so that the
// mask needs no second read of the values.  kFull: n == 32*W*R exactly.  On return gs->result is valid for
// every thread of the group.
template <int W, int R, bool kFull, bool kTable, typename KeyOf>
__device__ __forceinline__ void group_code_row(KeyOf keyof, int n, int tig, uint32_t* scratch, GroupShared* gs,
                                               int bar_id, const double* rcp, uint32_t (&kreg)[R]) {
  static_assert(W > 1, "single warps use warp_code_row");
  constexpr int GT = 32 * W;
  const int lane = tig & 31, warp = tig >> 5;
  const unsigned lt = (1u << lane) - 1u;
  const int first = warp * R * 32 + lane;

  uint32_t kmin = kPadKey, kmax = 0u;
  int cnt = 0;
#pragma unroll
  for (int k = 0; k < R; ++k) {
    uint32_t key = kZeroKey;
    const int i = first + k * 32;
    if (kFull || i < n) {
      key = keyof(i);
      kmin = min(kmin, key);
      kmax = max(kmax, key);
    }
    kreg[k] = key;
    cnt += __popc(__ballot_sync(0xFFFFFFFFu, key != kZeroKey));
  }
  kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
  kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
  if (lane == 0) {
    gs->wcnt[warp] = cnt;
    gs->wkmin[warp] = kmin;
    gs->wkmax[warp] = kmax;
  }
  group_barrier(bar_id, GT);
  int base = 0, m = 0;
#pragma unroll
  for (int w = 0; w < W; ++w) {
    const int c = gs->wcnt[w];
    if (w < warp) base += c;
    m += c;
    kmin = min(kmin, gs->wkmin[w]);
    kmax = max(kmax, gs->wkmax[w]);
  }
  // the non-zero keys of all warps, packed (their order is irrelevant)
#pragma unroll
  for (int k = 0; k < R; ++k) {
    const bool nz = kreg[k] != kZeroKey;
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, nz);
    if (nz) scratch[base + __popc(bal & lt)] = kreg[k];
    base += __popc(bal);
  }
  group_barrier(bar_id, GT);
  const bool bad = key_range_nonfinite(kmin, kmax);
  const int z = n - m;

  if (bad || kmin == kmax) {
    if (tig == 0) gs->result = trivial_row(bad, key_value(kmin));
  } else {
    const int per = (m + GT - 1) / GT;  // keys per thread needed
    if (per <= 4) group_sort_select<W, 4, kTable>(scratch, m, z, n, tig, gs, bar_id, rcp);
    else if (per <= 8) group_sort_select<W, 8, kTable>(scratch, m, z, n, tig, gs, bar_id, rcp);
    else if (per <= 16) group_sort_select<W, 16, kTable>(scratch, m, z, n, tig, gs, bar_id, rcp);
    else group_sort_select<W, 32, kTable>(scratch, m, z, n, tig, gs, bar_id, rcp);
  }
  group_barrier(bar_id, GT);
}

// Mask words of row `row` (of `rows`, ld words each, starting at `masks`) coded by a group: warp w produces words
// w*R .. w*R+R-1 (word w*R+k in lane k) and stores them with one coalesced write; words from W*R up to ld are
// written as 0.
template <int W, int R, bool kFull>
__device__ __forceinline__ void group_store_mask(const uint32_t (&kreg)[R], int n, int ld, int tig,
                                                 const RowResult& res, uint32_t* __restrict__ masks, int64_t row,
                                                 int64_t rows) {
  uint32_t* const out = masks + row * (int64_t)ld;
  const int lane = tig & 31, warp = tig >> 5;
  const bool flip = res.mode == 1;
  uint32_t mine = 0;
#pragma unroll
  for (int k = 0; k < R; ++k) {
    const int i = (warp * R + k) * 32 + lane;
    bool bit = (res.mode != 2) && (kFull || i < n) && ((kreg[k] >= res.tkey) != flip);
    uint32_t word = __ballot_sync(0xFFFFFFFFu, bit);
    if (lane == k) mine = word;
  }
  const int w = warp * R + lane;
  if (lane < R && w < ld && DAB_IN_BOUNDS(row * ld + w, rows * ld)) out[w] = mine;
  for (int p = W * R + tig; p < ld; p += 32 * W)
    if (DAB_IN_BOUNDS(row * ld + p, rows * ld)) out[p] = 0u;
}

// ---------------------------------------------------------------------------------------------------------
// One warp per row (rows of up to 32*R values).  The row's keys stay in registers (R per lane, element
// i = 32*k + lane in kreg[k]) so that the mask needs no second read of the values.
// ---------------------------------------------------------------------------------------------------------
template <int E>
__device__ __forceinline__ RowResult warp_sort_select(const uint32_t* scratch, int m, int z, int n, int lane,
                                                      const double* rcp) {
  uint32_t r[E];
#pragma unroll
  for (int j = 0; j < E; ++j) {
    int idx = j * 32 + lane;
    r[j] = idx < m ? scratch[idx] : kPadKey;
  }
  group_sort<1, E>(r, lane, nullptr, 0);
  return group_select<1, E, true>(r, m, z, n, lane, nullptr, 0, rcp);
}

// Rarely taken sizes (more than 256 non-zero keys) are kept out of line so that the registers of the common
// sizes set the occupancy.
template <int E>
__device__ __noinline__ RowResult warp_sort_select_outlined(const uint32_t* scratch, int m, int z, int n, int lane,
                                                            const double* rcp) {
  return warp_sort_select<E>(scratch, m, z, n, lane, rcp);
}

// Returns the result in every lane.  scratch: 32*R words of shared memory owned by the warp; rcp: n+1 reciprocals.
// kFull: n == 32*R exactly (no bounds tests in the load loop).
template <int R, bool kFull, typename KeyOf>
__device__ __forceinline__ RowResult warp_code_row(KeyOf keyof, int n, int lane, uint32_t* scratch,
                                                   const double* rcp, uint32_t (&kreg)[R]) {
  const unsigned lt = (1u << lane) - 1u;
  uint32_t kmin = kPadKey, kmax = 0u;
  int m = 0;
#pragma unroll
  for (int k = 0; k < R; ++k) {
    uint32_t key = kZeroKey;
    if (kFull || k * 32 < n) {
      const int i = k * 32 + lane;
      if (kFull || i < n) {
        key = keyof(i);
        kmin = min(kmin, key);
        kmax = max(kmax, key);
      }
      const bool nz = key != kZeroKey;
      const unsigned bal = __ballot_sync(0xFFFFFFFFu, nz);
      if (nz) scratch[m + __popc(bal & lt)] = key;  // the non-zero keys, in any order
      m += __popc(bal);
    }
    kreg[k] = key;
  }
  kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
  kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
  const bool bad = key_range_nonfinite(kmin, kmax);
  const int z = n - m;
  __syncwarp();

  RowResult res;
  if (bad || kmin == kmax) {
    res = trivial_row(bad, key_value(kmin));
  } else {
    const int per = (m + 31) >> 5;
    if (per <= 4) res = warp_sort_select<4>(scratch, m, z, n, lane, rcp);
    else if (per <= 8) res = warp_sort_select<8>(scratch, m, z, n, lane, rcp);
    else if (R <= 16 || per <= 16) res = warp_sort_select_outlined<16>(scratch, m, z, n, lane, rcp);
    else res = warp_sort_select_outlined<32>(scratch, m, z, n, lane, rcp);
    res.K = __shfl_sync(0xFFFFFFFFu, res.K, 0);
    res.alpha = __shfl_sync(0xFFFFFFFFu, res.alpha, 0);
    res.beta = __shfl_sync(0xFFFFFFFFu, res.beta, 0);
    res.flags = 0u;
    res.tkey = __shfl_sync(0xFFFFFFFFu, res.tkey, 0);
    res.mode = __shfl_sync(0xFFFFFFFFu, res.mode, 0);
  }
  __syncwarp();  // the scratch array may be overwritten by the next row
  return res;
}

// Mask words of the row from the keys in registers: word k in lane k (k < R), 0 elsewhere.
template <int R, bool kFull>
__device__ __forceinline__ uint32_t warp_mask_words(const uint32_t (&kreg)[R], int n, int lane, const RowResult& res) {
  uint32_t mine = 0;
  const bool flip = res.mode == 1;
#pragma unroll
  for (int k = 0; k < R; ++k) {
    // keys beyond n hold the zero key; they are masked here
    bool bit = (res.mode != 2) && (kFull || k * 32 + lane < n) && ((kreg[k] >= res.tkey) != flip);
    uint32_t word = __ballot_sync(0xFFFFFFFFu, bit);
    if (lane == k) mine = word;
  }
  return mine;
}

}  // namespace dab

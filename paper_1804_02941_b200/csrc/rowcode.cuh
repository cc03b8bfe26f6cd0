// Core of the row coder: a group of W warps turns one row of n fp32 values (read through an accessor
// from shared memory) into K, alpha, beta and the packed mask.
//
// Steps, all inside the group:
//   1. compaction  - keys of the non-zero values go to a scratch array; exact zeros are only counted.
//                    Equal values never straddle the best split, so the whole run of zeros is handled
//                    as one block of z elements with sum 0 at its place in the sorted order.
//   2. sort        - bitonic network on registers, E keys per thread, blocked layout (thread t owns
//                    sorted positions t*E .. t*E+E-1): strides below E stay inside a thread, strides
//                    below 32E use warp shuffles, larger ones go through shared memory.
//   3. scan        - fp64 running sums of the sorted values (thread-local, then across the group).
//   4. objective   - D_s of Algorithm 1 at every split between distinct values, arg-max with
//                    "largest s wins ties", done on (D, s) with integer reductions on the fp64 bits.
//   5. outputs     - orientation by |mean|, alpha/beta rounded once to fp32, threshold compare and
//                    ballot for the mask words.
#pragma once

#include "common.cuh"

namespace dab {

constexpr uint32_t kZeroKey = 0x80000000u;  // order_key(0.0f)

__device__ __forceinline__ void group_barrier(int bar_id, int threads) {
  if (threads == 32)
    __syncwarp();
  else
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(threads) : "memory");
}

// Skewed index into the scratch array: makes both the striped accesses of the compaction and the blocked
// accesses (stride E words between lanes, E a power of two up to 32) free of bank conflicts.
__device__ __forceinline__ int skew(int i) { return i + (i >> 5); }

template <int W, int E>
__device__ __forceinline__ void group_sort(uint32_t (&r)[E], int tig, uint32_t* xbuf, int bar_id) {
  constexpr int NTOT = 32 * W * E;
  const int ibase = tig * E;
#pragma unroll
  for (int k = 2; k <= NTOT; k <<= 1) {
#pragma unroll
    for (int st = k >> 1; st >= 1; st >>= 1) {
      if (st >= 32 * E) {  // partner lives in another warp: exchange through shared memory
        const bool up = (ibase & k) == 0;
        const bool lower = (ibase & st) == 0;
        const int partner = tig ^ (st / E);
#pragma unroll
        for (int j = 0; j < E; ++j) xbuf[j * (32 * W) + tig] = r[j];
        group_barrier(bar_id, 32 * W);
#pragma unroll
        for (int j = 0; j < E; ++j) {
          uint32_t o = xbuf[j * (32 * W) + partner];
          r[j] = (lower == up) ? min(r[j], o) : max(r[j], o);
        }
        group_barrier(bar_id, 32 * W);
      } else if (st >= E) {  // partner is another lane of this warp
        const bool up = (ibase & k) == 0;
        const bool lower = (ibase & st) == 0;
#pragma unroll
        for (int j = 0; j < E; ++j) {
          uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, r[j], st / E);
          r[j] = (lower == up) ? min(r[j], o) : max(r[j], o);
        }
      } else {  // both elements in this thread
#pragma unroll
        for (int j = 0; j < E; ++j) {
          if ((j & st) == 0) {
            uint32_t lo = min(r[j], r[j | st]), hi = max(r[j], r[j | st]);
            const bool up = (k < E) ? ((j & k) == 0) : ((ibase & k) == 0);
            r[j] = up ? lo : hi;
            r[j | st] = up ? hi : lo;
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
  uint32_t tkey;  // mask bit i = (key_i >= tkey) != low_side
  int mode;       // 0: e = [w >= t], 1: e = [w < t], 2: empty mask
};

struct GroupShared {   // per group, in shared memory
  double wsum[16];     // per-warp sums
  int wneg[16];        // per-warp counts of negative keys
  uint32_t wfirst[17]; // first key of each warp (index W: pad key)
  unsigned long long wbestD[16];
  int wbestS[16];
  double wbestP[16];
  uint32_t wbestT[16];
  int count;           // compaction counter
  int bad;             // non-finite seen
  int varied;          // two different keys seen
  RowResult result;
};

// Sorted keys in r[] (blocked), m real ones, z zeros elsewhere in the row, n row length.
template <int W, int E>
__device__ __forceinline__ void group_select(const uint32_t (&r)[E], int m, int z, int n, int tig, GroupShared* gs,
                                             int bar_id) {
  const int lane = tig & 31, warp = tig >> 5;
  const int q0 = tig * E;

  // thread-local sum and negative count
  double local = 0.0;
  int negc = 0;
#pragma unroll
  for (int j = 0; j < E; ++j) {
    if (q0 + j < m) {
      local = __dadd_rn(local, (double)key_value(r[j]));
      negc += (r[j] < kZeroKey);
    }
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
    group_barrier(bar_id, 32 * W);
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
  double excl = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
  if (lane == 0) excl = 0.0;
  double P = __dadd_rn(before, excl);

  // objective at every admissible split owned by this thread
  double bD = -1.0, bP = 0.0;
  int bS = 0;
  uint32_t bT = 0;
#pragma unroll
  for (int j = 0; j < E; ++j) {
    const int q = q0 + j;
    if (q < m) {
      const uint32_t kc = r[j];
      const uint32_t kn = (j + 1 < E) ? r[(j + 1 < E) ? j + 1 : j] : next_first;
      if (q == neg && z > 0) {  // split right after the block of zeros (low side: negatives and zeros)
        const int s = neg + z;
        if (s <= n - 1) {
          double D = objective(P, T, s, n);
          if (D >= bD) { bD = D; bP = P; bS = s; bT = kc; }
        }
      }
      P = __dadd_rn(P, (double)key_value(kc));
      const int s = (q < neg) ? q + 1 : q + 1 + z;
      const bool last = (q == m - 1);
      if (s <= n - 1 && (last || kc != kn)) {
        double D = objective(P, T, s, n);
        if (D >= bD) {
          bD = D; bP = P; bS = s;
          bT = (q == neg - 1 && z > 0) ? kZeroKey : kn;  // smallest value of the high side
        }
      }
    }
  }

  // arg-max of (D, s): D >= 0 (or -1 for "none"), so its bits order like a signed 64-bit integer
  long long dbits = __double_as_longlong(bD);
  int hi = (int)(dbits >> 32);
  int hmax = __reduce_max_sync(0xFFFFFFFFu, hi);
  unsigned lo = (hi == hmax) ? (unsigned)dbits : 0u;
  unsigned lmax = __reduce_max_sync(0xFFFFFFFFu, lo);
  bool top = (hi == hmax) && ((unsigned)dbits == lmax);
  int smax = __reduce_max_sync(0xFFFFFFFFu, top ? bS : -1);
  int src = __ffs(__ballot_sync(0xFFFFFFFFu, top && bS == smax)) - 1;
  bD = __shfl_sync(0xFFFFFFFFu, bD, src);
  bP = __shfl_sync(0xFFFFFFFFu, bP, src);
  bT = __shfl_sync(0xFFFFFFFFu, bT, src);
  bS = smax;
  if (W > 1) {
    if (lane == 0) {
      gs->wbestD[warp] = (unsigned long long)__double_as_longlong(bD);
      gs->wbestS[warp] = bS;
      gs->wbestP[warp] = bP;
      gs->wbestT[warp] = bT;
    }
    group_barrier(bar_id, 32 * W);
    if (tig == 0) {
      long long best = (long long)gs->wbestD[0];
      int bw = 0;
      for (int w = 1; w < W; ++w) {
        long long d = (long long)gs->wbestD[w];
        if (d > best || (d == best && gs->wbestS[w] > gs->wbestS[bw])) { best = d; bw = w; }
      }
      bS = gs->wbestS[bw];
      bP = gs->wbestP[bw];
      bT = gs->wbestT[bw];
    }
  }
  if (tig == 0) {
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
    gs->result = res;
  }
}

template <int W, int E>
__device__ __noinline__ void group_sort_select(uint32_t* scratch, int m, int z, int n, int tig, GroupShared* gs,
                                               int bar_id) {
  uint32_t r[E];
#pragma unroll
  for (int j = 0; j < E; ++j) {
    int idx = tig * E + j;
    r[j] = idx < m ? scratch[skew(idx)] : kPadKey;
  }
  if (W > 1) group_barrier(bar_id, 32 * W);  // scratch is reused for the cross-warp exchanges
  group_sort<W, E>(r, tig, scratch, bar_id);
  group_select<W, E>(r, m, z, n, tig, gs, bar_id);
}

// Codes one row.  `value(i)` returns element i (0 <= i < n) from shared memory.  On return gs->result is valid
// for every thread of the group (after the trailing barrier).
template <int W, typename Value>
__device__ __forceinline__ void group_code_row(Value value, int n, int tig, uint32_t* scratch, GroupShared* gs,
                                               int bar_id) {
  const int lane = tig & 31;
  constexpr int GT = 32 * W;
  if (W > 1) {
    if (tig == 0) {
      gs->count = 0;
      gs->bad = 0;
      gs->varied = 0;
    }
    group_barrier(bar_id, GT);
  }

  // 1. compaction of the non-zero keys (order within the scratch array is irrelevant)
  int bad = 0;
  int cnt = 0;             // W == 1: the warp's running count lives in a register
  uint32_t first_key = 0;  // any key of the row, to recognise constant rows
  for (int i0 = (tig >> 5) * 32; i0 < n; i0 += GT) {
    int i = i0 + lane;
    bool nz = false;
    uint32_t key = kZeroKey;
    if (i < n) {
      float x = value(i);
      bad |= is_nonfinite(x);
      key = order_key(x);
      nz = key != kZeroKey;
    }
    unsigned bal = __ballot_sync(0xFFFFFFFFu, nz);
    if (bal) {
      int base = cnt;
      if (W > 1) {
        if (lane == 0) base = atomicAdd(&gs->count, __popc(bal));
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
      } else {
        cnt += __popc(bal);
      }
      if (nz) scratch[skew(base + __popc(bal & ((1u << lane) - 1u)))] = key;
    }
  }
  bad = __any_sync(0xFFFFFFFFu, bad);
  int m = cnt;
  if (W > 1) {
    if (bad && lane == 0) gs->bad = 1;
    group_barrier(bar_id, GT);
    m = gs->count;
    bad = gs->bad;
  } else {
    __syncwarp();
  }
  const int z = n - m;

  // constant row: no non-zero at all, or no zero and all keys equal (checked after the sort would be
  // wasteful: compare every key with the first one instead)
  bool constant = (m == 0);
  if (!bad && !constant && z == 0) {
    first_key = scratch[skew(0)];
    int diff = 0;
    for (int i = tig; i < m; i += GT) diff |= (scratch[skew(i)] != first_key);
    diff = __any_sync(0xFFFFFFFFu, diff);
    if (W > 1) {
      if (diff && lane == 0) gs->varied = 1;
      group_barrier(bar_id, GT);
      constant = (gs->varied == 0);
    } else {
      constant = !diff;
    }
  }

  if (bad || constant) {
    if (tig == 0) {
      RowResult res;
      res.K = 0;
      float c = bad ? __uint_as_float(0x7FC00000u) : (m == 0 ? 0.0f : key_value(first_key));
      res.alpha = c;
      res.beta = c;
      res.flags = bad ? DAB_ROW_NONFINITE : DAB_ROW_DEGENERATE;
      res.tkey = 0u;
      res.mode = 2;
      gs->result = res;
    }
  } else {
    const int per = (m + GT - 1) / GT;  // keys per thread needed
    if (per <= 4) group_sort_select<W, 4>(scratch, m, z, n, tig, gs, bar_id);
    else if (per <= 8) group_sort_select<W, 8>(scratch, m, z, n, tig, gs, bar_id);
    else if (per <= 16) group_sort_select<W, 16>(scratch, m, z, n, tig, gs, bar_id);
    else group_sort_select<W, 32>(scratch, m, z, n, tig, gs, bar_id);
  }
  group_barrier(bar_id, GT);
}

}  // namespace dab

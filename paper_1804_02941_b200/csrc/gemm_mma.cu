// Tensor-core form of the AND-popcount contraction (Section 4.2: the four population counts of a pair of
// coded rows).  popc(e AND f) over a row of n bits is the dot product of the two rows written as 0/1 bytes,
// so each CTA expands mask words to bytes in shared memory and lets the fifth-generation tensor cores
// (tcgen05.mma, kind::i8, 32-bit integer accumulators in tensor memory) form a 128 x NT block of exact integer
// counts.  The bytes are 0 / -1 (signed operands on both sides: one byte permutation per four bits makes them,
// and (-1) x (-1) = 1), in an order of the row's bits that is permuted within each word, alike on both sides.  The four-term rescale then runs on the counts as they are read
// back from tensor memory, with the same arithmetic as the population-count kernel.
//
// Shared-memory operand layout (K-major, no swizzle): 8 rows x 16 bytes form one contiguous 128-byte core
// matrix; core matrices of consecutive 16-byte K chunks follow each other (leading byte offset 128) and
// groups of 8 rows are one whole stage row apart (stride byte offset = K chunks per stage x 128).  One mask
// word is 32 K bytes = two K chunks = the K extent of one kind::i8 instruction.
#include <algorithm>

#include "common.cuh"
#include "tc.cuh"

namespace dab {
namespace {

using namespace tc;

__device__ unsigned int g_mma_wait_timeouts;

constexpr int MMA_M = tc::kLanes;  // activation rows per CTA = lanes of tensor memory
constexpr int MMA_NMAX = 256;      // weight rows per CTA = columns of tensor memory

// One operand of the contraction: packed rows with their popcounts and the two reconstruction values
// (gamma, delta on the activation side; alpha, beta on the weight side).
struct Side {
  const uint32_t* mask;
  int32_t ld;
  const int32_t* K;
  const float* v1;  // value of the set bits
  const float* v0;  // value of the clear bits
  int64_t rows;
};

// What the epilogue needs of one column-side row: its two values, its popcount K and n - K as doubles, and
// its part of the output offset.
struct __align__(16) ColumnParams {
  double v1, v0, K, nK;
  int64_t off;
  int64_t pad;
};

// The pieces one thread expands per stage: unit u covers row (u>>3)/KQ*8 + (u&7), 16-byte piece (u>>3)%KQ.
// Eight consecutive lanes hold the eight rows of one core matrix, so their 16-byte stores are one
// contiguous 128 bytes; their loads read KQ x 16 contiguous bytes per row.
//
// One CTA forms one 128 x NT tile over the whole row length, 4*KQ mask words per stage.  There is a single
// stage: a CTA alternates between expanding and waiting for the tensor cores, and the overlap comes from the
// several CTAs resident on an SM (expansion, the fp64 rescale and the tensor pipe use different units), which
// measured faster than two stages with fewer resident CTAs.
//
// kLanesAreActivations: the rows that ride the 128 lanes of tensor memory (and the threads of the epilogue)
// are activation rows, the columns weight rows: coalesced stores when the output is contiguous along the
// activation rows (NCHW).  Otherwise the roles are exchanged: coalesced for a row-major M x N output.
template <int THREADS, int KQ, int MIN_CTAS, int NT_MAX, bool kLanesAreActivations>
__global__ void __launch_bounds__(THREADS, MIN_CTAS) binary_gemm_mma_kernel(const GemmArgs g, const int tile_cols) {
  constexpr int KC = 8 * KQ;            // 16-byte K chunks per stage (two per mask word)
  constexpr uint32_t SBO = KC * 128;    // bytes between groups of 8 rows
  constexpr int kMaxUnits = ((MMA_M + NT_MAX) * KQ + THREADS - 1) / THREADS;  // NT <= NT_MAX in this shape
  extern __shared__ __align__(128) unsigned char dyn_mem[];  // [lane-side stage][column-side stage][ColumnParams]
  __shared__ __align__(8) uint64_t s_bar;
  __shared__ uint32_t s_tmem;

  const Side act{g.A, g.lda, g.KA, g.gamma, g.delta, g.M}, wgt{g.B, g.ldb, g.KB, g.alpha, g.beta, g.N};
  const Side L = kLanesAreActivations ? act : wgt;  // lane side
  const Side S = kLanesAreActivations ? wgt : act;  // column side

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t i0 = (int64_t)blockIdx.x * MMA_M;
  const int64_t j0 = (int64_t)blockIdx.y * tile_cols;        // tile_cols: 64, 128 or 256 column-side rows per CTA
  const int nrows = (int)min((int64_t)tile_cols, S.rows - j0);  // column-side rows of this tile
  const int NT = (nrows + 15) & ~15;                            // instruction N
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < NT) tmem_cols <<= 1;

  const uint32_t a_bytes = MMA_M * KC * 16;
  const int ncap = (int)min((int64_t)tile_cols, (S.rows + 15) & ~(int64_t)15);  // widest tile of this launch
  const uint32_t mem0 = (smem_u32(dyn_mem) + 127u) & ~127u;
  unsigned char* const stage = dyn_mem + (mem0 - smem_u32(dyn_mem));
  ColumnParams* const s_col = reinterpret_cast<ColumnParams*>(stage + a_bytes + (uint32_t)ncap * KC * 16);
  const uint32_t bar = smem_u32(&s_bar);

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // where activation row i and weight row j meet in the output: act_offset(i) + j * col_stride
  auto act_offset = [&](int64_t i) {
    return (i / g.map.inner) * g.map.outer_stride + (i % g.map.inner) * g.map.row_stride;
  };
  for (int j = tid; j < nrows; j += THREADS) {
    ColumnParams cp;
    const int K = S.K[DAB_IDX(j0 + j, S.rows)];
    cp.v1 = (double)S.v1[DAB_IDX(j0 + j, S.rows)];
    cp.v0 = (double)S.v0[DAB_IDX(j0 + j, S.rows)];
    cp.K = (double)K;
    cp.nK = (double)(g.n - K);
    cp.off = kLanesAreActivations ? (j0 + j) * g.map.col_stride : act_offset(j0 + j);
    cp.pad = 0;
    s_col[j] = cp;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = s_tmem;
  const uint32_t idesc = instr_desc(NT, true, true);  // both operands signed: bytes 0 / -1

  // units of this thread: lane-side pieces first, then column-side pieces
  const int l_units = MMA_M * KQ, units = l_units + NT * KQ;
  const int chunks = (g.words + 4 * KQ - 1) / (4 * KQ);
  const int real_words = (g.n + 31) >> 5;  // words beyond these hold no bits
  uint4 q[kMaxUnits];

  auto fetch = [&](int c) {  // the 16-byte pieces of chunk c, zero beyond the operands
    const int w0 = c * 4 * KQ;
#pragma unroll
    for (int t = 0; t < kMaxUnits; ++t) {
      const int u = tid + t * THREADS;
      q[t] = make_uint4(0, 0, 0, 0);
      if (u >= units) continue;
      const bool isL = u < l_units;
      const int v = isL ? u : u - l_units;
      const int row = ((v >> 3) / KQ) * 8 + (v & 7), piece = (v >> 3) % KQ;
      const int w = w0 + 4 * piece;
      if (w >= g.words) continue;
      if (isL) {
        if (i0 + row < L.rows)
          q[t] = *reinterpret_cast<const uint4*>(L.mask + DAB_IDX((i0 + row) * (int64_t)L.ld + w, L.rows * L.ld - 3));
      } else {
        if (row < nrows)
          q[t] = *reinterpret_cast<const uint4*>(S.mask + DAB_IDX((j0 + row) * (int64_t)S.ld + w, S.rows * S.ld - 3));
      }
    }
  };

  bool dead = false;
  uint32_t parity = 0;
  fetch(0);
  for (int c = 0; c < chunks; ++c) {
    if (c > 0) {  // the instructions that read the stage for the previous chunk have completed
      mbar_wait(bar, parity, dead, &g_mma_wait_timeouts);
      parity ^= 1;
    }
#pragma unroll
    for (int t = 0; t < kMaxUnits; ++t) {
      const int u = tid + t * THREADS;
      if (u >= units) continue;
      const bool isL = u < l_units;
      const int v = isL ? u : u - l_units;
      const int group = (v >> 3) / KQ, piece = (v >> 3) % KQ;
      if (c * 4 * KQ + 4 * piece >= g.words) continue;  // no instruction reads this part of the stage
      unsigned char* dst =
          stage + (isL ? 0u : a_bytes) + (uint32_t)group * SBO + (uint32_t)(8 * piece) * 128 + (v & 7) * 16;
      expand_words_signed(q[t], dst);
    }
    if (c + 1 < chunks) fetch(c + 1);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy stores -> tensor-core reads
    __syncthreads();
    if (tid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t a_addr = mem0, b_addr = mem0 + a_bytes;
      const int kw = min(4 * KQ, real_words - c * 4 * KQ);
      for (int t = 0; t < kw; ++t)  // one mask word = 32 K bytes = two K chunks per instruction
        mma_i8(tmem, smem_desc(a_addr + t * 256, 128, SBO), smem_desc(b_addr + t * 256, 128, SBO), idesc,
               (c | t) != 0);
      mma_commit(bar);
    }
  }
  mbar_wait(bar, parity, dead, &g_mma_wait_timeouts);  // the last commit covers every instruction issued before it
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

  // Epilogue: thread = lane-side row (a warp reads the 32 lanes of its quarter), 32 columns at a time.
  {
    const int64_t gl = i0 + (warp & 3) * 32 + lane;
    const bool valid = gl < L.rows && !dead;
    double Kl = 0.0, l1 = 0.0, l0 = 0.0;
    int64_t off = 0;
    if (valid) {
      Kl = (double)L.K[DAB_IDX(gl, L.rows)];
      l1 = (double)L.v1[DAB_IDX(gl, L.rows)];
      l0 = (double)L.v0[DAB_IDX(gl, L.rows)];
      off = kLanesAreActivations ? act_offset(gl) : gl * g.map.col_stride;
    }
    const bool want_p11 = g.p11 != nullptr;
    float* const crow = g.C + off;
    // this row's counts: element (gl, j0 + j) when the lanes are activation rows, (j0 + j, gl) otherwise
    const int64_t p0 = kLanesAreActivations ? gl * g.ldp + j0 : j0 * g.ldp + gl;
    const int64_t pstep = kLanesAreActivations ? 1 : g.ldp;
    for (int cb = warp >> 2; cb * 32 < NT; cb += THREADS / 128) {
      uint32_t v[32];
      tmem_load_32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(cb * 32), v);
      if (!valid) continue;
      const int left = nrows - cb * 32;  // columns of this block that exist
      const ColumnParams* const col = s_col + cb * 32;
      const int64_t pblock = p0 + (int64_t)(cb * 32) * pstep;
#pragma unroll
      for (int jj = 0; jj < 32; ++jj) {
        if (jj >= left) break;
        const ColumnParams cp = col[jj];
        // The four counts as doubles (small integers: every difference is exact, so these are the values
        // rescale() converts from int), then its four terms in its order: alpha gamma p11, alpha delta p10,
        // beta gamma p01, beta delta p00, with p10 the count on the weight side only.
        const double p11 = int_to_double((int)v[jj]);
        const double pc = __dsub_rn(cp.K, p11), pl = __dsub_rn(Kl, p11);  // set on the column / lane side only
        const double p00 = __dsub_rn(cp.nK, pl);
        double y = __dmul_rn(__dmul_rn(cp.v1, l1), p11);
        if (kLanesAreActivations) {
          y = __dadd_rn(y, __dmul_rn(__dmul_rn(cp.v1, l0), pc));
          y = __dadd_rn(y, __dmul_rn(__dmul_rn(cp.v0, l1), pl));
        } else {
          y = __dadd_rn(y, __dmul_rn(__dmul_rn(l1, cp.v0), pl));
          y = __dadd_rn(y, __dmul_rn(__dmul_rn(l0, cp.v1), pc));
        }
        y = __dadd_rn(y, __dmul_rn(__dmul_rn(cp.v0, l0), p00));
        if (DAB_IN_BOUNDS(off + cp.off, g.c_extent)) crow[cp.off] = (float)y;
        if (want_p11 && DAB_IN_BOUNDS(pblock + jj * pstep, (g.M - 1) * g.ldp + g.N)) g.p11[pblock + jj * pstep] = (int)v[jj];
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
}

inline size_t dynamic_bytes(int kq, int ncap) {
  return (size_t)(MMA_M + ncap) * (8 * kq) * 16 + (size_t)ncap * sizeof(ColumnParams) + 128;
}

template <int THREADS, int KQ, int MIN_CTAS, int NT_MAX, bool kLanesAreActivations>
cudaError_t launch_shape(const GemmArgs& args, dim3 grid, int tile_cols, int ncap, cudaStream_t stream) {
  auto kernel = binary_gemm_mma_kernel<THREADS, KQ, MIN_CTAS, NT_MAX, kLanesAreActivations>;
  cudaError_t e = ensure_dynamic_smem(kernel, dynamic_bytes(KQ, NT_MAX));
  if (e != cudaSuccess) return e;
  kernel<<<grid, THREADS, dynamic_bytes(KQ, ncap), stream>>>(args, tile_cols);
  return cudaGetLastError();
}

template <bool kLanesAreActivations>
cudaError_t launch_side(const GemmArgs& args, cudaStream_t stream) {
  const int64_t lane_rows = kLanesAreActivations ? args.M : args.N, col_rows = kLanesAreActivations ? args.N : args.M;
  // Column tile: the full 256 columns of an accumulator unless that leaves most SMs without a CTA.
  const int64_t gx = (lane_rows + MMA_M - 1) / MMA_M;
  int tile_cols = MMA_NMAX;
  while (tile_cols > 64 && gx * ((col_rows + tile_cols - 1) / tile_cols) < 2 * sm_count()) tile_cols >>= 1;
  const int64_t gy = (col_rows + tile_cols - 1) / tile_cols;
  if (gx > 0x7FFFFFFF || gy > 65535) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)gx, (unsigned)gy);
  const int ncap = (int)std::min<int64_t>(tile_cols, (col_rows + 15) & ~(int64_t)15);
  // CTA shape by tile width, from timings of the four layer shapes of the ResNet-18-like stack: narrow tiles
  // run best as many small CTAs (six of 128 threads per SM), wider ones as fewer CTAs of 256 threads with
  // longer stages (two per SM at the full 256 columns, where shared memory is the limit).
  if (ncap <= 64) return launch_shape<128, 1, 6, 64, kLanesAreActivations>(args, grid, tile_cols, ncap, stream);
  if (ncap <= 128 && args.words >= 64)  // long rows: eight words per stage halve the dependent stage rounds
    return launch_shape<256, 2, 3, 128, kLanesAreActivations>(args, grid, tile_cols, ncap, stream);
  if (ncap <= 128) return launch_shape<256, 1, 4, 128, kLanesAreActivations>(args, grid, tile_cols, ncap, stream);
  return launch_shape<256, 2, 2, MMA_NMAX, kLanesAreActivations>(args, grid, tile_cols, ncap, stream);
}

}  // namespace

cudaError_t launch_gemm_mma(const GemmArgs& args, bool lanes_along_rows, cudaStream_t stream) {
  if (args.words < 1 || args.M < 1 || args.N < 1) return cudaErrorInvalidValue;
  return lanes_along_rows ? launch_side<true>(args, stream) : launch_side<false>(args, stream);
}

cudaError_t read_mma_wait_timeouts(unsigned int* count) {
  return cudaMemcpyFromSymbol(count, g_mma_wait_timeouts, sizeof(unsigned int));
}

}  // namespace dab

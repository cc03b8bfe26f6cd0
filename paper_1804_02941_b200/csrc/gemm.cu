// dab_binary_gemm: AND-popcount contraction of packed rows with the four-term rescale fused in.
// Integer work (AND, carry-save adders, POPC, IADD); the only large byte stream is the output store.
#include "common.cuh"

namespace dab {

constexpr int BM = 64, BN = 64;  // tile of outputs
constexpr int BK = 48;           // words per staged slice (a multiple of 3 for the carry-save groups and of 4)
constexpr int TM = 4, TN = 4;    // outputs per thread
constexpr int GEMM_THREADS = 256;
constexpr int SLD = BM + 4;      // padded smem row, keeps 16-byte alignment

// Population counts issue at a quarter of the rate of logic operations, so three AND-ed words are first
// compressed by a carry-save adder (two 3-input logic operations) into a sum word and a carry word:
// popc(x0) + popc(x1) + popc(x2) = popc(sum) + 2 popc(carry).  Two counts instead of three.
__device__ __forceinline__ void csa(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t& sum, uint32_t& carry) {
  asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(sum) : "r"(x0), "r"(x1), "r"(x2));    // x0 ^ x1 ^ x2
  asm("lop3.b32 %0, %1, %2, %3, 0xE8;" : "=r"(carry) : "r"(x0), "r"(x1), "r"(x2));  // majority
}

// kLanesAlongRows: consecutive threads own consecutive activation rows i (coalesced when the output is
// contiguous along i, as in NCHW); otherwise consecutive threads own consecutive weight columns j.
template <bool kLanesAlongRows>
__global__ void __launch_bounds__(GEMM_THREADS) binary_gemm_kernel(const GemmArgs g) {
  __shared__ __align__(16) uint32_t As[BK][SLD];
  __shared__ __align__(16) uint32_t Bs[BK][SLD];

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int a_t = kLanesAlongRows ? tx : ty;  // which group of TM activation rows
  const int b_t = kLanesAlongRows ? ty : tx;  // which group of TN weight rows
  const int64_t i0 = (int64_t)blockIdx.x * BM;
  const int64_t j0 = (int64_t)blockIdx.y * BN;

  int ones[TM][TN], twos[TM][TN];  // p11 = ones + 2 * twos
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) ones[i][j] = twos[i][j] = 0;

  for (int k0 = 0; k0 < g.words; k0 += BK) {
    // stage BK words of 64 rows of each operand, transposed; words beyond the row length become 0
#pragma unroll
    for (int rep = 0; rep < (BM * BK / 4) / GEMM_THREADS; ++rep) {
      const int t = tid + rep * GEMM_THREADS;
      const int r = t / (BK / 4), q = (t % (BK / 4)) * 4;
      uint4 qa = make_uint4(0, 0, 0, 0), qb = make_uint4(0, 0, 0, 0);
      if (k0 + q < g.words) {
        if (i0 + r < g.M)
          qa = *reinterpret_cast<const uint4*>(g.A + DAB_IDX((i0 + r) * (int64_t)g.lda + k0 + q, g.M * g.lda - 3));
        if (j0 + r < g.N)
          qb = *reinterpret_cast<const uint4*>(g.B + DAB_IDX((j0 + r) * (int64_t)g.ldb + k0 + q, g.N * g.ldb - 3));
      }
      As[q + 0][r] = qa.x; As[q + 1][r] = qa.y; As[q + 2][r] = qa.z; As[q + 3][r] = qa.w;
      Bs[q + 0][r] = qb.x; Bs[q + 1][r] = qb.y; Bs[q + 2][r] = qb.z; Bs[q + 3][r] = qb.w;
    }
    __syncthreads();
    const int kw = min(BK, g.words - k0);
    const int groups = (kw + 2) / 3;  // the slice is zero-filled up to BK, a multiple of 3
#pragma unroll 1
    for (int gq = 0; gq < groups; ++gq) {
      const int w = gq * 3;
      uint32_t av[3][TM], bv[3][TN];
#pragma unroll
      for (int t = 0; t < 3; ++t) {
        uint4 a = *reinterpret_cast<const uint4*>(&As[w + t][a_t * TM]);
        uint4 b = *reinterpret_cast<const uint4*>(&Bs[w + t][b_t * TN]);
        av[t][0] = a.x; av[t][1] = a.y; av[t][2] = a.z; av[t][3] = a.w;
        bv[t][0] = b.x; bv[t][1] = b.y; bv[t][2] = b.z; bv[t][3] = b.w;
      }
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) {
          uint32_t sum, carry;
          csa(av[0][i] & bv[0][j], av[1][i] & bv[1][j], av[2][i] & bv[2][j], sum, carry);
          ones[i][j] += __popc(sum);
          twos[i][j] += __popc(carry);
        }
    }
    __syncthreads();
  }

  double al[TN], be[TN];
  int Ke[TN];
#pragma unroll
  for (int j = 0; j < TN; ++j) {
    int64_t gj = j0 + b_t * TN + j;
    const bool in = gj < g.N;
    al[j] = in ? (double)g.alpha[DAB_IDX(gj, g.N)] : 0.0;
    be[j] = in ? (double)g.beta[DAB_IDX(gj, g.N)] : 0.0;
    Ke[j] = in ? g.KB[DAB_IDX(gj, g.N)] : 0;
  }
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    int64_t gi = i0 + a_t * TM + i;
    if (gi >= g.M) continue;
    int Kf = g.KA[DAB_IDX(gi, g.M)];
    double gam = (double)g.gamma[DAB_IDX(gi, g.M)], del = (double)g.delta[DAB_IDX(gi, g.M)];
    int64_t base = (gi / g.map.inner) * g.map.outer_stride + (gi % g.map.inner) * g.map.row_stride;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      int64_t gj = j0 + b_t * TN + j;
      if (gj >= g.N) continue;
      int p11 = ones[i][j] + 2 * twos[i][j];
      if (DAB_IN_BOUNDS(base + gj * g.map.col_stride, g.c_extent))
        g.C[base + gj * g.map.col_stride] = rescale(p11, Ke[j], Kf, g.n, al[j], be[j], gam, del);
      if (g.p11 && DAB_IN_BOUNDS(gi * g.ldp + gj, (g.M - 1) * g.ldp + g.N)) g.p11[gi * g.ldp + gj] = p11;
    }
  }
}

cudaError_t launch_gemm(const GemmArgs& args, bool lanes_along_rows, cudaStream_t stream) {
  dim3 grid((unsigned)((args.M + BM - 1) / BM), (unsigned)((args.N + BN - 1) / BN));
  if (grid.y > 65535) return cudaErrorInvalidValue;
  if (lanes_along_rows)
    binary_gemm_kernel<true><<<grid, GEMM_THREADS, 0, stream>>>(args);
  else
    binary_gemm_kernel<false><<<grid, GEMM_THREADS, 0, stream>>>(args);
  return cudaGetLastError();
}


}  // namespace dab

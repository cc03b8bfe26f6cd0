// dab_binary_gemm: AND-popcount contraction of packed rows with the four-term rescale fused in.
// Integer work (AND, POPC, IADD) on the ALU pipes; the only large byte stream is the output store.
#include "common.cuh"

namespace dab {

constexpr int BM = 64, BN = 64, BK = 32;  // tile of outputs, words per staged slice
constexpr int TM = 4, TN = 4;             // outputs per thread
constexpr int GEMM_THREADS = 256;
constexpr int SLD = BM + 4;               // padded smem row, keeps 16-byte alignment

// Four-term rescale in fp64, one rounding to fp32.  Term order is part of the contract.
__device__ __forceinline__ float rescale(int p11, int Ke, int Kf, int n, double a, double b, double g, double d) {
  int p10 = Ke - p11, p01 = Kf - p11, p00 = n - Ke - Kf + p11;
  double y = __dmul_rn(__dmul_rn(a, g), (double)p11);
  y = __dadd_rn(y, __dmul_rn(__dmul_rn(a, d), (double)p10));
  y = __dadd_rn(y, __dmul_rn(__dmul_rn(b, g), (double)p01));
  y = __dadd_rn(y, __dmul_rn(__dmul_rn(b, d), (double)p00));
  return (float)y;
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

  int acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0;

  const int lrow = tid >> 3;        // 0..31
  const int lquad = (tid & 7) * 4;  // word offset inside the slice

  for (int k0 = 0; k0 < g.words; k0 += BK) {
#pragma unroll
    for (int rep = 0; rep < 2; ++rep) {
      int r = lrow + rep * 32;
      uint4 qa = make_uint4(0, 0, 0, 0), qb = make_uint4(0, 0, 0, 0);
      if (k0 + lquad < g.words) {
        if (i0 + r < g.M) qa = *reinterpret_cast<const uint4*>(g.A + (i0 + r) * (int64_t)g.lda + k0 + lquad);
        if (j0 + r < g.N) qb = *reinterpret_cast<const uint4*>(g.B + (j0 + r) * (int64_t)g.ldb + k0 + lquad);
      }
      As[lquad + 0][r] = qa.x; As[lquad + 1][r] = qa.y; As[lquad + 2][r] = qa.z; As[lquad + 3][r] = qa.w;
      Bs[lquad + 0][r] = qb.x; Bs[lquad + 1][r] = qb.y; Bs[lquad + 2][r] = qb.z; Bs[lquad + 3][r] = qb.w;
    }
    __syncthreads();
#pragma unroll 8
    for (int w = 0; w < BK; ++w) {
      uint4 a = *reinterpret_cast<const uint4*>(&As[w][a_t * TM]);
      uint4 b = *reinterpret_cast<const uint4*>(&Bs[w][b_t * TN]);
      uint32_t av[TM] = {a.x, a.y, a.z, a.w};
      uint32_t bv[TN] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] += __popc(av[i] & bv[j]);
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < TM; ++i) {
    int64_t gi = i0 + a_t * TM + i;
    if (gi >= g.M) continue;
    int Kf = g.KA[gi];
    double gam = (double)g.gamma[gi], del = (double)g.delta[gi];
    int64_t base = (gi / g.map.inner) * g.map.outer_stride + (gi % g.map.inner) * g.map.row_stride;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      int64_t gj = j0 + b_t * TN + j;
      if (gj >= g.N) continue;
      int p11 = acc[i][j];
      g.C[base + gj * g.map.col_stride] =
          rescale(p11, g.KB[gj], Kf, g.n, (double)g.alpha[gj], (double)g.beta[gj], gam, del);
      if (g.p11) g.p11[gi * g.ldp + gj] = p11;
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

// Measurement aid: independent AND + POPC + IADD chains, 16 per thread per round.
__global__ void __launch_bounds__(256) popc_probe_kernel(uint32_t* sink, int iters) {
  uint32_t a[4], b[4];
  int acc[16];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    a[i] = 0x9E3779B9u * (threadIdx.x + 1 + i);
    b[i] = 0x85EBCA6Bu * (blockIdx.x + 7 + i);
  }
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = 0;
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i * 4 + j] += __popc(a[i] & b[j]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // change the operands so that nothing can be hoisted out of the loop
      a[i] = a[i] * 1664525u + 1013904223u;
      b[i] ^= a[i] >> 7;
    }
  }
  int s = 0;
#pragma unroll
  for (int i = 0; i < 16; ++i) s += acc[i];
  sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = (uint32_t)s;
}

cudaError_t launch_popc_probe(uint32_t* sink, int32_t blocks, int32_t iters, cudaStream_t stream) {
  popc_probe_kernel<<<blocks, 256, 0, stream>>>(sink, iters);
  return cudaGetLastError();
}

}  // namespace dab

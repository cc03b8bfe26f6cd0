// Inline-PTX helpers shared by the tensor-core kernels: shared-memory and instruction descriptors of
// tcgen05.mma kind::i8, bounded mbarrier waits, tensor-memory loads and the expansion of mask bits to bytes.
//
// Shared-memory operand layout used throughout (K-major, no swizzle): 8 rows x 16 bytes form one contiguous
// 128-byte core matrix; core matrices of consecutive 16-byte K chunks follow each other (leading byte offset
// 128) and groups of 8 rows are one whole stage row apart (stride byte offset = K chunks per stage x 128).
// One kind::i8 instruction covers 32 K bytes = two K chunks.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace dab {
namespace tc {

constexpr int kLanes = 128;                      // rows of an accumulator = lanes of tensor memory
constexpr long long kWaitCycles = 4000000000ll;  // about two seconds; a wait that long has failed

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Shared-memory matrix descriptor: address, leading and stride byte offsets in 16-byte units, descriptor
// version 1 in bits [46,48), no swizzle (layout type 0 in bits [61,64)).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
         ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46);
}

// Instruction descriptor of kind::i8: D format S32 (2 at bit 4), A format at bit 7 and B format at bit 10
// (0: unsigned 8-bit, 1: signed 8-bit), both K-major (0 at bits 15 and 16), N / 8 at bit 17, M / 16 at bit 24.
__device__ __forceinline__ uint32_t instr_desc(int nt, bool a_signed = false, bool b_signed = false) {
  return (2u << 4) | ((a_signed ? 1u : 0u) << 7) | ((b_signed ? 1u : 0u) << 10) | ((uint32_t)(nt >> 3) << 17) |
         ((uint32_t)(kLanes >> 4) << 24);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// Bounded wait for the phase with the given parity.  Returns false after `limit` cycles and counts the failure
// in *failures (device global); the caller then stops waiting on anything (dead stays set) but keeps its
// control flow, so that every thread still reaches every barrier and the CTA ends.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, bool& dead, unsigned int* failures,
                                          long long limit = kWaitCycles) {
  if (dead) return false;
  const long long t0 = clock64();
  for (;;) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    if (clock64() - t0 > limit) {
      dead = true;
      atomicAdd(failures, 1u);
      return false;
    }
  }
}

__device__ __forceinline__ void mma_i8(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
      :
      : "r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
      : "memory");
}

// Arrives on the barrier once every tcgen05.mma issued by this thread so far has completed.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem_addr, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem_addr), "r"(cols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t tmem, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(cols) : "memory");
}

__device__ __forceinline__ void tmem_load_32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Eight consecutive columns of this warp's 32 lanes (no wait: follow with tmem_load_wait).
__device__ __forceinline__ void tmem_load_8(uint32_t taddr, uint32_t (&v)[8]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
      : "r"(taddr)
      : "memory");
}

__device__ __forceinline__ void tmem_load_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Four mask bits -> four bytes of 0/1 (bit i to byte i): the products i + 7j land on distinct bit positions.
__device__ __forceinline__ uint32_t spread4(uint32_t nibble) { return (nibble * 0x00204081u) & 0x01010101u; }

// One 16-byte piece (four mask words) of one row -> eight 16-byte K chunks in the stage.
// dst points at the row's slot in the K chunk of the first word; consecutive K chunks are 128 bytes apart.
__device__ __forceinline__ void expand_words(uint4 q, unsigned char* dst) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int m = 0; m < 4; ++m) {
    uint4 lo, hi;
    lo.x = spread4(w[m] & 15u);
    lo.y = spread4((w[m] >> 4) & 15u);
    lo.z = spread4((w[m] >> 8) & 15u);
    lo.w = spread4((w[m] >> 12) & 15u);
    hi.x = spread4((w[m] >> 16) & 15u);
    hi.y = spread4((w[m] >> 20) & 15u);
    hi.z = spread4((w[m] >> 24) & 15u);
    hi.w = spread4(w[m] >> 28);
    *reinterpret_cast<uint4*>(dst + (2 * m) * 128) = lo;
    *reinterpret_cast<uint4*>(dst + (2 * m + 1) * 128) = hi;
  }
}

// Four mask bits -> four bytes of 0 / -1 with one byte permutation: the selector's nibbles are bits s, s+4, s+8
// and s+12 of the word shifted right by s (their lowest bit picks byte 0x00 or 0xFF of the source; the other
// selector bits pick among copies of the same two bytes, and sign replication of 0x00 / 0xFF changes nothing).
__device__ __forceinline__ uint32_t select4(uint32_t selector) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %1, %2;" : "=r"(d) : "r"(0xFF00FF00u), "r"(selector));
  return d;
}

// One 16-byte piece (four mask words) of one row -> eight 16-byte K chunks of 0 / -1 bytes (signed 8-bit
// operands: (-1) x (-1) = 1, so the integer dot product of two such rows is popc(e AND f)).  Within a word's
// 32 bytes the bits appear in the order 0 4 8 12, 1 5 9 13, 2 6 10 14, 3 7 11 15, then the same for the upper
// half: a permutation of the contraction index, the same on both operands, that the sum does not see.
__device__ __forceinline__ void expand_words_signed(uint4 q, unsigned char* dst) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int m = 0; m < 4; ++m) {
    uint4 lo, hi;
    lo.x = select4(w[m]);
    lo.y = select4(w[m] >> 1);
    lo.z = select4(w[m] >> 2);
    lo.w = select4(w[m] >> 3);
    hi.x = select4(w[m] >> 16);
    hi.y = select4(w[m] >> 17);
    hi.z = select4(w[m] >> 18);
    hi.w = select4(w[m] >> 19);
    *reinterpret_cast<uint4*>(dst + (2 * m) * 128) = lo;
    *reinterpret_cast<uint4*>(dst + (2 * m + 1) * 128) = hi;
  }
}

}  // namespace tc
}  // namespace dab

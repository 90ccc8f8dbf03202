// tcgen05 building blocks of the Stage-1 proxy GEMV (Sec. 4.1 proxy equations, Sec. 4.3 Stage 1).
//
// The packed proxy rows are the A operand of an integer tensor-core MMA exactly as they lie in memory:
//   D[m][n] += sum_k A[k][m] * B[k][n],  A = bytes of 32 kept proxy rows (u8, 128 bytes of each row: M = 128),
//   B = the inputs x_k of those rows as signed base-256 digits (s8), D = int32 accumulators in tensor memory.
// A is "MN-major" (a row of the proxy is contiguous along M), in the 128-byte-swizzled shared-memory
// layout: row k of a 32-row stage lives at (k / 8) * 1024 + (k % 8) * 128, and its 16-byte chunk c at
// position c ^ (k % 8).  B is MN-major without swizzle, 16 columns: row k is the 16 bytes at k * 16.
// A byte of a 4-bit proxy holds two codes (16 * hi + lo); a second MMA over the bytes with the high nibble
// masked off gives the lo sums, the difference the hi sums.  Integer products and sums are exact.
#pragma once

#include <stdint.h>

namespace prox {

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// One warp allocates all 512 columns (one block per SM owns the tensor memory) and frees them again.
__device__ __forceinline__ void tmem_alloc_all(uint32_t result_smem_addr) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(result_smem_addr), "r"(512u) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free_all(uint32_t taddr) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(512u) : "memory");
}

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all in units of 16
// bytes), descriptor version 1, swizzle mode (0 none, 2 = 128 bytes).
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo, uint32_t swizzle) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)swizzle << 61);
}
// Instruction descriptor of kind::i8: int32 accumulate, A unsigned, B signed, both MN-major, M x N.
__device__ __forceinline__ constexpr uint32_t umma_idesc_u8s8(int M, int N) {
  return (2u << 4) | (0u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
      :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u) : "memory");
}
// The mbarrier gets one arrival when every MMA this thread issued before has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 16 consecutive 32-bit columns of the warp's 32 lanes (lane l of the warp = data path lane base + l)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st16_zero(uint32_t taddr) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
               :: "r"(taddr), "r"(0u) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// A bf16 input as an integer times a power of two shared by the call: x = X * 2^(ebase - 134), with
// ebase = max(largest biased exponent - 22, 1), so |X| < 2^30 (inputs more than 22 binades below the
// largest lose low bits: below 2^-24 of the result).  Returned as four signed base-256 digits
// (byte d = digit d, each in [-128, 127], X = sum digit_d 256^d).
__device__ __forceinline__ uint32_t x_digits(uint32_t bf16_bits, int ebase) {
  const int E = (int)((bf16_bits >> 7) & 0xffu);
  const int m = (int)(bf16_bits & 0x7fu) | (E ? 0x80 : 0);
  const int sh = (E > 1 ? E : 1) - ebase;
  int X = sh >= 0 ? (m << sh) : (sh > -9 ? ((m + (1 << (-sh - 1))) >> (-sh)) : 0);
  if (bf16_bits & 0x8000u) X = -X;
  return ((uint32_t)X + 0x00808080u) ^ 0x00808080u;
}
// sum_d digit_d 256^d of int32 digit sums, in fp32 (every digit sum is far below 2^31)
__device__ __forceinline__ float digits_to_float(uint32_t d0, uint32_t d1, uint32_t d2, uint32_t d3) {
  float v = (float)(int)d3;
  v = fmaf(v, 256.f, (float)(int)d2);
  v = fmaf(v, 256.f, (float)(int)d1);
  return fmaf(v, 256.f, (float)(int)d0);
}

}  // namespace prox

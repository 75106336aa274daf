// tcgen05 building blocks shared by the tensor-memory scan kernels (scan_fwd_tc.cu, scan_bwd_tc.cu):
// shared-memory and instruction descriptors, MMA issue, commit, tensor-memory loads and stores.
#pragma once

#include <stdint.h>

#include "pipeline.cuh"

namespace m2rnn {

// K-major, 128-byte-swizzled canonical layout (rows of 128 bytes = 64 bf16, groups of 8 rows 1024
// bytes apart, the 16-byte chunks of a row XOR-ed with the row index modulo 8).
//   bits  0-13 start address >> 4     bits 32-45 stride between 8-row groups >> 4
//   bits 16-29 leading offset >> 4 (unused by swizzled K-major layouts)
//   bits 46-47 descriptor version 1   bits 61-63 swizzle mode (2 = 128 bytes)
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t sa) {
  return (uint64_t)((sa & 0x3ffffu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// The same with 64-byte swizzling (mode 4): rows of 64 bytes = 32 bf16, groups of 8 rows 512 bytes
// apart, the 16-byte chunks of a row XOR-ed with (row / 2) modulo 4.  Serves both readings of such a
// tile: K-major (a row = one M/N index, 32 K indices) and MN-major (a row = one K index, 32 M/N
// indices); the instruction descriptor's major bits say which.
__device__ __forceinline__ uint64_t smem_desc_sw64(uint32_t sa) {
  return (uint64_t)((sa & 0x3ffffu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(512 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)4 << 61);
}
// Instruction descriptor of kind::f16 with bf16 operands: fp32 accumulator (bits 4-5 = 1), bf16 A
// and B (bits 7-9 and 10-12 = 1), both K-major (bits 15, 16 = 0), N >> 3 in bits 17-22, M >> 4 in
// bits 24-28.
__host__ __device__ constexpr uint32_t idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[128 x N] (+)= A[128 x 16] B[N x 16]^T: A from tensor memory (lane = row, 8 columns of two bf16),
// B from shared memory
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit_tc(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n .reg .pred p;\n elect.sync _|p, 0xffffffff;\n selp.u32 %0, 1, 0, p;\n}" : "=r"(pred));
  return pred != 0;
}
// 8 or 16 consecutive 32-bit columns of this warp's 32 lanes
__device__ __forceinline__ void tmem_ld(uint32_t taddr, float (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
               : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld(uint32_t taddr, float (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7]), "=f"(r[8]),
        "=f"(r[9]), "=f"(r[10]), "=f"(r[11]), "=f"(r[12]), "=f"(r[13]), "=f"(r[14]), "=f"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}


// Operands read "MN-major": a tile stored [k][m] with m contiguous (rows of 128 bytes = 64 elements
// along M or N, eight rows = one 1024-byte swizzle atom along K).  Leading offset = distance between
// the 64-element blocks along M/N, stride = distance between 8-row groups along K.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t sa, uint32_t lead_bytes) {
  return (uint64_t)((sa & 0x3ffffu) >> 4) | ((uint64_t)((lead_bytes & 0x3ffffu) >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// kind::f16, bf16 operands, fp32 accumulator, A and B MN-major (bits 15 and 16)
__host__ __device__ constexpr uint32_t idesc_bf16_mn(int M, int N) { return idesc_bf16(M, N) | (1u << 15) | (1u << 16); }
// D[128 x N] (+)= A B^T with both operands from shared memory
__device__ __forceinline__ void umma_bf16_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

}  // namespace m2rnn

// Helpers for the kernels that drive the 5th-generation tensor cores directly (tcgen05.mma with operands in shared
// memory and the accumulator in tensor memory): operand and instruction descriptors, issue, commit, bounded waits.
#pragma once
#include <stdint.h>
#include <cuda_bf16.h>

namespace umma {

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
// Shared-memory operand descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(const void* smem_ptr) {
  const uint64_t addr = (uint64_t)(smem_u32(smem_ptr) & 0x3FFFF) >> 4;
  uint64_t d = addr;                       // bits [0,14): start address / 16
  d |= (uint64_t)1 << 16;                  // bits [16,30): leading-dimension byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;        // bits [32,46): stride between 8-row groups / 16
  d |= (uint64_t)1 << 46;                  // bits [46,48): descriptor version of this architecture
  d |= (uint64_t)2 << 61;                  // bits [61,64): 128-byte swizzle
  return d;
}
// Shared-memory operand descriptor: K-major without swizzle.  Core matrices are 8 rows x 16 bytes, stored contiguously
// (128 bytes); lbo = bytes between core matrices adjacent along K, sbo = bytes between core matrices adjacent along M/N.
__device__ __forceinline__ uint64_t umma_desc_nosw(const void* smem_ptr, unsigned lbo, unsigned sbo) {
  uint64_t d = (uint64_t)(smem_u32(smem_ptr) & 0x3FFFF) >> 4;
  d |= (uint64_t)(lbo >> 4) << 16;
  d |= (uint64_t)(sbo >> 4) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}
// byte offset of element (row r, k) of an [R x 32] bf16 operand in that layout (core matrices of one K chunk contiguous)
__device__ __forceinline__ size_t nosw_offset(int R, int r, int k) {
  return (size_t)(k >> 3) * ((size_t)(R >> 3) * 128) + (size_t)(r >> 3) * 128 + (size_t)(r & 7) * 16 + (size_t)(k & 7) * 2;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, N and M.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
// bounded wait on an mbarrier phase; false when the iteration budget runs out
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity) {
  for (int it = 0; it < 20000000; ++it) {
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}
// Shared-memory operand descriptor for the SAME 128-byte-swizzled tile read the other way round (MN-major): the tile
// holds rows of 128 channels as two 64-channel halves (rows x 128 bytes each, 16-byte chunks XOR-swizzled by the row
// number); as an operand whose M (or N) index is the channel and whose K index is the row, its atoms are 64 channels x
// 8 rows.  lbo = bytes between the two 64-channel halves, sbo = bytes between groups of 8 rows (1024).  A K step of 16
// rows advances the start address by 2048 bytes.  (Checked against a host product with a stand-alone probe.)
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(const void* smem_ptr, unsigned lbo, unsigned sbo) {
  uint64_t d = (uint64_t)(smem_u32(smem_ptr) & 0x3FFFF) >> 4;
  d |= (uint64_t)(lbo >> 4) << 16;
  d |= (uint64_t)(sbo >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// byte offset of 16-byte chunk `ch` (0..15) of row `r` inside a [rows x 128 channels] bf16 operand tile:
// two column blocks of 64 channels (128 bytes per row each), chunks XOR-swizzled by the row number
__device__ __forceinline__ size_t sw128_offset(int rows, int r, int ch) {
  return (size_t)(ch >> 3) * ((size_t)rows * 128) + (size_t)r * 128 + (size_t)(((ch & 7) ^ (r & 7)) << 4);
}

constexpr uint32_t kIdescAMnMajor = 1u << 15;              // instruction descriptor: operand A is MN-major

}  // namespace umma

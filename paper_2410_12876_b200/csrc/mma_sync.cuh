// Warp-level pieces shared by the kernels whose contraction has a small M (2..16 rows): 16-byte
// asynchronous copies into shared memory, ldmatrix, and the m16n8k16 bf16 MMA with its fragment
// layouts (PTX ISA, "Matrix fragments for mma.m16n8k16").  With g = lane / 4, t = lane % 4:
//   A (16 x 16, row-major): a0 = (row g, cols 2t, 2t+1), a1 = (row g+8, same), a2 = (row g, cols 2t+8, 2t+9), a3 = (row g+8, same)
//   B (16 x 8, column-major): b0 = (rows 2t, 2t+1, col g), b1 = (rows 2t+8, 2t+9, col g)
//   C (16 x 8): c0, c1 = (row g, cols 2t, 2t+1), c2, c3 = (row g+8, same)
#pragma once
#include "ag_common.cuh"

namespace ag {

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void *gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16 x 8, f32) += A (16 x 16, bf16, row-major fragments) * B (16 x 8, bf16, column-major fragments)
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
// Byte offset of 16-byte piece `piece` (0..15) of row `row` in a shared-memory tile of 256-byte rows
// (128 bf16): pieces are XOR-ed with the row number so that the eight rows one ldmatrix reads fall
// into different banks.
__device__ __forceinline__ uint32_t tile256_off(int row, int piece) {
  return (uint32_t)(row * 256 + ((piece ^ (row & 7)) << 4));
}

}  // namespace ag

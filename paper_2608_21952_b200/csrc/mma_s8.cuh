// Warp-level int8 tile product on shared-memory operands whose rows are contiguous along
// the contraction axis (A[m][k], B[n][k]); int32 accumulation is exact.
#pragma once
#include "common.cuh"

namespace ssdi8 {

__device__ __forceinline__ void mma_m16n8k32_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// acc[nt][4] += A[row0 .. row0+15][0 .. K) * B[n0 + 8 nt .. +7][0 .. K)^T for nt < NT.
// lda / ldb are row strides in bytes (multiples of 4).  Accumulator element e of tile nt is
// (row = row0 + lane/4 + 8 (e/2), col = n0 + 8 nt + 2 (lane%4) + (e%2)).
template <int NT>
__device__ __forceinline__ void warp_gemm_s8(int (&acc)[NT][4], const int8_t* A, int lda, int row0,
                                             const int8_t* B, int ldb, int n0, int K) {
  const int lane = threadIdx.x & 31, gq = lane >> 2, tq = lane & 3;
  const int8_t* a_lo = A + (size_t)(row0 + gq) * lda + tq * 4;
  const int8_t* a_hi = a_lo + 8 * (size_t)lda;
  for (int k0 = 0; k0 < K; k0 += 32) {
    const uint32_t a0 = *reinterpret_cast<const uint32_t*>(a_lo + k0);
    const uint32_t a1 = *reinterpret_cast<const uint32_t*>(a_hi + k0);
    const uint32_t a2 = *reinterpret_cast<const uint32_t*>(a_lo + k0 + 16);
    const uint32_t a3 = *reinterpret_cast<const uint32_t*>(a_hi + k0 + 16);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int8_t* bp = B + (size_t)(n0 + 8 * nt + gq) * ldb + tq * 4 + k0;
      const uint32_t b0 = *reinterpret_cast<const uint32_t*>(bp);
      const uint32_t b1 = *reinterpret_cast<const uint32_t*>(bp + 16);
      mma_m16n8k32_s8(acc[nt], a0, a1, a2, a3, b0, b1);
    }
  }
}

}  // namespace ssdi8

// ChunkBMM on the group axis (Section 4.2): acc_cb[i,j] = sum_n Cq[i,n] Bq[j,n] per
// (batch, chunk, group), INT32 exact, then one INT32 -> INT8 step
//   CBq = rne(fmul(float(acc_cb), fdiv(fmul(s_C, s_B), s_cb))).
// Only 64 x 64 tiles that touch the causal half (tile column <= tile row) are computed.
#include "kernels.h"
#include "mma_s8.cuh"

namespace ssdi8 {
namespace {

constexpr int TB = 64;  // tile edge

__global__ void __launch_bounds__(128) bmm_kernel(const int8_t* __restrict__ Cq,
                                                  const int8_t* __restrict__ Bq,
                                                  const float* __restrict__ s_C,
                                                  const float* __restrict__ s_B,
                                                  const float* __restrict__ s_cb,
                                                  int8_t* __restrict__ CBq,
                                                  int32_t* __restrict__ tap_acc,
                                                  uint32_t* __restrict__ absmax_acc, Dims d) {
  extern __shared__ __align__(16) int8_t smem[];
  const int nt = d.Q / TB;
  // blockIdx.x enumerates the lower-triangular tiles (ti >= tj)
  int ti = 0, rem = blockIdx.x;
  while (rem > ti) { rem -= ti + 1; ++ti; }
  const int tj = rem;
  (void)nt;
  const int g = blockIdx.y % d.G;
  const int bk = blockIdx.y / d.G;  // b * c + k
  const int N = d.N, ld = N + 16;
  int8_t* Cs = smem;
  int8_t* Bs = smem + TB * ld;
  const i64 tok0 = (i64)bk * d.Q;  // b*L + k*Q
  const int w4 = N / 4;
  for (int e = threadIdx.x; e < TB * w4; e += blockDim.x) {
    const int r = e / w4, w = e % w4;
    *reinterpret_cast<uint32_t*>(Cs + r * ld + 4 * w) =
        *reinterpret_cast<const uint32_t*>(Cq + ((tok0 + ti * TB + r) * d.G + g) * N + 4 * w);
    *reinterpret_cast<uint32_t*>(Bs + r * ld + 4 * w) =
        *reinterpret_cast<const uint32_t*>(Bq + ((tok0 + tj * TB + r) * d.G + g) * N + 4 * w);
  }
  __syncthreads();
  int acc[8][4];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[a][e] = 0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  warp_gemm_s8<8>(acc, Cs, ld, warp * 16, Bs, ld, 0, N);
  const float r_cb = s_cb ? __fdiv_rn(__fmul_rn(s_C[g], s_B[g]), s_cb[g]) : 0.f;
  const i64 base = ((i64)bk * d.G + g) * d.Q * d.Q;
  int amax = 0;
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int i = ti * TB + warp * 16 + (lane >> 2) + 8 * (e >> 1);
      const int j = tj * TB + 8 * a + 2 * (lane & 3) + (e & 1);
      const i64 o = base + (i64)i * d.Q + j;
      if (tap_acc) tap_acc[o] = acc[a][e];
      if (CBq) CBq[o] = (int8_t)rne_clamp(__fmul_rn((float)acc[a][e], r_cb));
      if (j <= i) amax = max(amax, abs(acc[a][e]));
    }
  if (absmax_acc) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if (lane == 0) atomicMax(absmax_acc + g, (uint32_t)amax);
  }
}

}  // namespace

ssdi8_status_t launch_bmm(const Dims& d, const int8_t* Cq, const int8_t* Bq, const float* s_C,
                          const float* s_B, const float* s_cb, int8_t* CBq, int32_t* tap_acc,
                          uint32_t* absmax_acc, cudaStream_t st) {
  const int nt = d.Q / TB;
  dim3 grid(nt * (nt + 1) / 2, d.b * d.c * d.G);
  size_t smem = 2 * TB * (d.N + 16);
  bmm_kernel<<<grid, 128, smem, st>>>(Cq, Bq, s_C, s_B, s_cb, s_cb ? CBq : nullptr, tap_acc,
                                      absmax_acc, d);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

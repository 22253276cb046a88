// ChunkState with the sparse-aware reformulation (Eq. 3) and the INT32 rescale (Eq. 4):
//   LUT_state[i] = fmul(dt_i, exp32(fsub(cs_last, cs_i)))
//   Xs_q[i,p]    = rne(fmul(fmul(float(xq[i,p]), fdiv(s_x, s_xs)), LUT_state[i]))
//   acc_st[p,n]  = sum_i Xs_q[i,p] Bq[i,n]   (contraction over the tokens of the chunk)
//   loc[p,n]     = fmul(float(acc_st), fmul(s_xs[h,p], s_B[g]))
// One block per (batch, chunk, head).
#include "kernels.h"
#include "mma_s8.cuh"

namespace ssdi8 {
namespace {

__global__ void __launch_bounds__(256) chunk_state_kernel(
    const int8_t* __restrict__ xq, const int8_t* __restrict__ Bq, const float* __restrict__ s_x,
    const float* __restrict__ s_xs, const float* __restrict__ s_B, const float* __restrict__ dt,
    const float* __restrict__ cs, float* __restrict__ loc, int8_t* __restrict__ tap_Xsq,
    int32_t* __restrict__ tap_acc, uint32_t* __restrict__ absmax_xs, Dims d) {
  extern __shared__ __align__(16) int8_t smem[];
  const int Q = d.Q, P = d.P, N = d.N, ld = Q + 16;
  const int h = blockIdx.x, k = blockIdx.y, b = blockIdx.z;
  const int g = h / (d.H / d.G);
  int8_t* XsT = smem;                  // [P][ld]  Xs_q transposed: row p, token contiguous
  int8_t* BT = smem + P * ld;          // [N][ld]
  float* lut = reinterpret_cast<float*>(smem + (P + N) * ld);  // [Q]
  const i64 tok0 = (i64)b * d.L + (i64)k * Q;
  const float* csk = cs + (((i64)b * d.H + h) * d.c + k) * Q;
  const float cs_last = csk[Q - 1];
  for (int i = threadIdx.x; i < Q; i += blockDim.x)
    lut[i] = __fmul_rn(dt[(tok0 + i) * d.H + h], exp32(__fsub_rn(cs_last, csk[i])));
  __syncthreads();
  // --- prologue: X_scaled, re-quantised, written transposed
  const int pw = P / 4;  // words per token
  const int pq = threadIdx.x % pw;
  float rx[4], sx[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    sx[u] = s_x[h * P + 4 * pq + u];
    rx[u] = absmax_xs ? sx[u] : __fdiv_rn(sx[u], s_xs[h * P + 4 * pq + u]);
  }
  float mx[4] = {0.f, 0.f, 0.f, 0.f};
  for (int i = threadIdx.x / pw; i < Q; i += blockDim.x / pw) {
    const i64 o = ((tok0 + i) * d.H + h) * P + 4 * pq;
    const uint32_t w = *reinterpret_cast<const uint32_t*>(xq + o);
    const float l = lut[i];
    if (absmax_xs) {
#pragma unroll
      for (int u = 0; u < 4; ++u)
        mx[u] = fmaxf(mx[u], fabsf(__fmul_rn(__fmul_rn((float)sx8(w, u), rx[u]), l)));
    } else {
      int q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        q[u] = rne_clamp(__fmul_rn(__fmul_rn((float)sx8(w, u), rx[u]), l));
        XsT[(4 * pq + u) * ld + i] = (int8_t)q[u];
      }
      if (tap_Xsq) *reinterpret_cast<uint32_t*>(tap_Xsq + o) = pack4(q[0], q[1], q[2], q[3]);
    }
  }
  if (absmax_xs) {
#pragma unroll
    for (int u = 0; u < 4; ++u) atomicMax(absmax_xs + h * P + 4 * pq + u, __float_as_uint(mx[u]));
    return;
  }
  const int nw = N / 4;
  for (int e = threadIdx.x; e < Q * nw; e += blockDim.x) {
    const int i = e / nw, w4 = e % nw;
    const uint32_t w = *reinterpret_cast<const uint32_t*>(Bq + ((tok0 + i) * d.G + g) * N + 4 * w4);
#pragma unroll
    for (int u = 0; u < 4; ++u) BT[(4 * w4 + u) * ld + i] = (int8_t)sx8(w, u);
  }
  __syncthreads();
  // --- acc[p][n]: 8 warps = 4 row blocks of 16 p  x  2 column halves of N/2
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = (warp & 3) * 16, nh = N / 2, n0 = (warp >> 2) * nh;
  const float sB = s_B[g];
  const i64 obase = ((((i64)b * d.c + k) * d.H + h) * P) * N;
  for (int nb = 0; nb < nh; nb += 32) {
    int acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[a][e] = 0;
    warp_gemm_s8<4>(acc, XsT, ld, row0, BT, ld, n0 + nb, Q);
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int p = row0 + (lane >> 2) + 8 * (e >> 1);
        const int n = n0 + nb + 8 * a + 2 * (lane & 3) + (e & 1);
        const i64 o = obase + (i64)p * N + n;
        if (tap_acc) tap_acc[o] = acc[a][e];
        loc[o] = __fmul_rn((float)acc[a][e], __fmul_rn(s_xs[h * P + p], sB));
      }
  }
}

}  // namespace

ssdi8_status_t launch_chunk_state(const Dims& d, const int8_t* xq, const int8_t* Bq,
                                  const float* s_x, const float* s_xs, const float* s_B,
                                  const float* dt, const float* cs, float* loc, int8_t* tap_Xsq,
                                  int32_t* tap_acc, uint32_t* absmax_xs, cudaStream_t st) {
  dim3 grid(d.H, d.c, d.b);
  size_t smem = (size_t)(d.P + d.N) * (d.Q + 16) + sizeof(float) * d.Q;
  static bool attr_done = false;
  if (!attr_done) {
    SSDI8_CUDA_CHECK(cudaFuncSetAttribute(chunk_state_kernel,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024));
    attr_done = true;
  }
  chunk_state_kernel<<<grid, 256, smem, st>>>(xq, Bq, s_x, s_xs, s_B, dt, cs, loc, tap_Xsq, tap_acc,
                                              absmax_xs, d);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

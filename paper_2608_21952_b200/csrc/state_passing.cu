// StatePassing (Eq. 5-6; Algorithm 2 module 3) on fp32 states:
//   S_k = fmaf(Gamma_k, S_{k-1}, loc_k);  prev[k] = S_{k-1};  hq[k] = rne(fmul(S_{k-1}, 1/s_h))
// The only sequential loop of the layer (over chunks); everything else is parallel over
// (b, h, p, n).  HBM-bound: each thread owns 4 consecutive n (16-byte loads of loc, 4-byte
// packed stores of hq) and keeps several chunk loads in flight.
#include "kernels.h"

namespace ssdi8 {
namespace {

constexpr int SP_T = 256;

__global__ void __launch_bounds__(SP_T) state_passing_kernel(
    const float4* loc /* may alias prev: no __restrict__ */, const float* __restrict__ gamma, const float4* __restrict__ init,
    const float* __restrict__ s_h, float4* prev, float4* __restrict__ final_state,
    uint32_t* __restrict__ hq, uint32_t* __restrict__ absmax_h, Dims d) {
  const int N4 = d.N / 4;
  const i64 per_b = (i64)d.H * d.P * N4;               // float4 per (b) slice of one chunk
  const i64 idx = (i64)blockIdx.x * SP_T + threadIdx.x;  // over b * H * P * N4
  if (idx >= per_b * d.b) return;
  const int b = (int)(idx / per_b);
  const i64 r = idx % per_b;                             // (h, p, n4)
  const int hp = (int)(r / N4);                          // h * P + p
  const int h = hp / d.P;
  float inv_h = 0.f;
  if (hq) inv_h = __fdiv_rn(1.0f, s_h[hp]);
  float4 S = init ? init[idx] : make_float4(0.f, 0.f, 0.f, 0.f);
  const float* gm = gamma + ((i64)b * d.H + h) * d.c;
  float m = 0.f;
  const i64 stride = per_b;                              // chunk stride in float4
  i64 o = (i64)b * d.c * per_b + r;
  for (int k = 0; k < d.c; ++k, o += stride) {
    const float4 l = loc[o];  // read before prev[o] is written: prev may alias loc
    const float g = gm[k];
    if (hq)
      hq[o] = pack4(rne_clamp(__fmul_rn(S.x, inv_h)), rne_clamp(__fmul_rn(S.y, inv_h)),
                    rne_clamp(__fmul_rn(S.z, inv_h)), rne_clamp(__fmul_rn(S.w, inv_h)));
    if (prev) prev[o] = S;
    if (absmax_h) m = fmaxf(fmaxf(fmaxf(m, fabsf(S.x)), fmaxf(fabsf(S.y), fabsf(S.z))), fabsf(S.w));
    S.x = __fmaf_rn(g, S.x, l.x);
    S.y = __fmaf_rn(g, S.y, l.y);
    S.z = __fmaf_rn(g, S.z, l.z);
    S.w = __fmaf_rn(g, S.w, l.w);
  }
  if (final_state) final_state[idx] = S;
  if (absmax_h) {
    m = fmaxf(fmaxf(fmaxf(m, fabsf(S.x)), fmaxf(fabsf(S.y), fabsf(S.z))), fabsf(S.w));
    // lanes of a warp that share (h,p): N4 consecutive threads (N4 = 16 or 32)
    for (int off = 1; off < N4 && off < 32; off <<= 1)
      m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if ((threadIdx.x & (min(N4, 32) - 1)) == 0) atomicMax(absmax_h + hp, __float_as_uint(m));
  }
}

}  // namespace

ssdi8_status_t launch_state_passing(const Dims& d, const float* loc, const float* gamma,
                                    const float* init, const float* s_h, float* prev,
                                    float* final_state, int8_t* hq, uint32_t* absmax_h,
                                    cudaStream_t st) {
  const i64 n = (i64)d.b * d.H * d.P * (d.N / 4);
  unsigned grid = (unsigned)((n + SP_T - 1) / SP_T);
  state_passing_kernel<<<grid, SP_T, 0, st>>>(
      reinterpret_cast<const float4*>(loc), gamma, reinterpret_cast<const float4*>(init), s_h,
      reinterpret_cast<float4*>(prev), reinterpret_cast<float4*>(final_state),
      reinterpret_cast<uint32_t*>(hq), absmax_h, d);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

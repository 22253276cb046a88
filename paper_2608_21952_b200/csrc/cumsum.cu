// ChunkCumsum (Algorithm 2, module 1) and the per-token scalars every later module derives
// from it.  For each (batch, head, chunk) it writes one contiguous pack of 6 rows of Q floats:
//   row 0  cs[i]    = (float) sum_{i'<=i} (double)dt (double)A_h, in token order   (dA_cs)
//   row 1  dt[i]
//   row 2  woff[i]  = fmul(dt_i, exp32(fsub(cs_ie, cs_i))), ie = last token of i's 16-token sub-block
//   row 3  atok[i]  = exp32(fsub(cs_i, cs_{i-1}))  (1 for i = 0): the per-token decay
//   row 4  bounds that let the scan kernel skip sub-blocks that cannot matter (they decide no
//          output bit): [c] = fmul(127, wmax_c), wmax_c the maximum of |woff| over the 16-token
//          sub-block c; [16 + c] = the maximum of the former over sub-blocks 0..c, times
//          1.00001, or +inf when cs is not non-increasing over the chunk (some dt A > 0), which
//          switches the early exits of the scan kernel off; entries from 32 on are not written
//   row 5  lut[i]   = fmul(dt_i, exp32(fsub(cs_last, cs_i)))                       (LUT_state)
// and Gamma[b,h,k] = exp32(cs[Q-1]) (Decay_pass, Eq. 5).  The sum order is part of the definition
// (it decides rounding downstream), so each (b, chunk, head) is scanned sequentially by one
// thread; loads and stores go through shared memory so that the [b,L,H] reads and the row
// writes coalesce.  Later kernels fetch a pack with one bulk copy and need no exponentials
// per token.
#include "kernels.h"

namespace ssdi8 {
namespace {

constexpr int CH = 8;  // heads per block

__global__ void __launch_bounds__(256) cumsum_kernel(const float* __restrict__ dt,
                                                     const float* __restrict__ A,
                                                     float* __restrict__ pack,
                                                     float* __restrict__ gamma,
                                                     float* __restrict__ tap_cs, Dims d) {
  extern __shared__ float tile[];  // dt [CH][Q+1], cs [CH][Q+1], woff [CH][Q+1]
  const int Q = d.Q, ld = Q + 1;
  const int lq = 31 - __clz(Q);  // Q is a power of two
  float* dts = tile;
  float* css = tile + CH * ld;
  float* wos = tile + 2 * CH * ld;
  const int h0 = blockIdx.x * CH, k = blockIdx.y, b = blockIdx.z;
  const int nh = min(CH, d.H - h0);
  const i64 t0 = (i64)b * d.L + (i64)k * Q;
  // (all loads of a round of 8 before the first store: the loads are the latency of this phase)
  for (int e0 = threadIdx.x; e0 < Q * CH; e0 += 8 * blockDim.x) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + u * blockDim.x;
      const int i = e / CH, hh = e % CH;
      v[u] = (e < Q * CH && hh < nh) ? __ldg(dt + (t0 + i) * d.H + h0 + hh) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + u * blockDim.x;
      const int i = e / CH, hh = e % CH;
      if (e < Q * CH && hh < nh) dts[hh * ld + i] = v[u];
    }
  }
  __syncthreads();
  if (threadIdx.x < nh) {
    const int hh = threadIdx.x;
    const double a = (double)A[h0 + hh];
    double acc = 0.0;
    float last = 0.f;
    float dmin = 0.f, dmax = 0.f;  // every increment dt A <= 0  <=>  no dt has the sign of A
    // Q is a multiple of 8: loads and products (exact in binary64) of 8 tokens are independent,
    // only the additions form the chain
    for (int i0 = 0; i0 < Q; i0 += 8) {
      float dv[8];
      double pr[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        dv[j] = dts[hh * ld + i0 + j];
        pr[j] = (double)dv[j] * a;
        dmin = fminf(dmin, dv[j]);
        dmax = fmaxf(dmax, dv[j]);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        acc += pr[j];
        last = (float)acc;
        css[hh * ld + i0 + j] = last;
      }
    }
    const bool mono = a > 0.0 ? dmax <= 0.f : (a < 0.0 ? dmin >= 0.f : true);
    css[hh * ld + Q] = mono ? 1.0f : 0.0f;
    gamma[((i64)b * d.H + h0 + hh) * d.c + k] = exp32(last);
  }
  __syncthreads();
  const i64 u0 = ((i64)b * d.H + h0) * d.c + k;  // pack index of head h0; the next head is d.c further
  for (int e = threadIdx.x; e < Q * CH; e += blockDim.x) {
    const int hh = e >> lq, i = e & (Q - 1);
    if (hh >= nh) continue;
    const float* c = css + hh * ld;
    const float ci = c[i], di = dts[hh * ld + i];
    const i64 u = u0 + (i64)hh * d.c;
    float* p = pack + ((u * kPackRows) << lq) + i;
    p[0] = ci;
    p[Q] = di;
    const float wo = __fmul_rn(di, exp32(__fsub_rn(c[i | 15], ci)));
    wos[hh * ld + i] = wo;
    p[PACK_WOFF * Q] = wo;
    p[PACK_ATOK * Q] = i > 0 ? exp32(__fsub_rn(ci, c[i - 1])) : 1.0f;
    p[PACK_LUT * Q] = __fmul_rn(di, exp32(__fsub_rn(c[Q - 1], ci)));
    if (tap_cs) tap_cs[(u << lq) + i] = ci;
  }
  __syncthreads();
  // sub-block maxima of |woff| (dts is free now: it holds them, times 127)
  for (int e = threadIdx.x; e < CH * 16; e += blockDim.x) {
    const int hh = e >> 4, c = e & 15;
    if (hh >= nh || c >= Q / 16) continue;
    float m = 0.f;
    for (int j = 0; j < 16; ++j) m = fmaxf(m, fabsf(wos[hh * ld + c * 16 + j]));
    dts[hh * ld + c] = __fmul_rn(127.0f, m);
  }
  __syncthreads();
  for (int e = threadIdx.x; e < 32 * CH; e += blockDim.x) {   // the first 32 entries of the bounds row
    const int hh = e >> 5, i = e & 31;
    if (hh >= nh) continue;
    float m = 0.f;
    if (i < Q / 16) {
      m = dts[hh * ld + i];
    } else if (i >= 16 && i < 16 + Q / 16) {
      for (int c = 0; c <= i - 16; ++c) m = fmaxf(m, dts[hh * ld + c]);
      m = css[hh * ld + Q] != 0.f ? __fmul_rn(m, 1.00001f) : __int_as_float(0x7f800000);
    }
    pack[(((u0 + (i64)hh * d.c) * kPackRows + PACK_WMAX) << lq) + i] = m;
  }
}

}  // namespace

ssdi8_status_t launch_cumsum(const Dims& d, const float* dt, const float* A, float* pack,
                             float* gamma, float* tap_cs, cudaStream_t st) {
  dim3 grid((d.H + CH - 1) / CH, d.c, d.b);
  size_t smem = sizeof(float) * 3 * CH * (d.Q + 1);
  cumsum_kernel<<<grid, 256, smem, st>>>(dt, A, pack, gamma, tap_cs, d);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

// Shared device helpers of the SSDi8 kernels: the binary32 building blocks that
// decide integer codes (never contracted, never approximated) and small utilities.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ssdi8.h"

namespace ssdi8 {

typedef long long i64;

// round half to even, saturate to [-127, 127] (Eq. 1: 2^(b-1)-1 levels per side)
__device__ __forceinline__ int rne_clamp(float v) {
  float r = rintf(v);
  r = fmaxf(r, -127.0f);  // fmaxf(NaN, a) = a
  r = fminf(r, 127.0f);
  return __float2int_rn(r);
}

// binary32 exponential with a fixed operation sequence (see ssdi8.h): Cody-Waite
// reduction by ln 2, degree-7 Taylor polynomial (Horner, fmaf), scaling by 2^n
// through the exponent field.  0 below -80, argument clamped at +80.
__device__ __forceinline__ float exp32(float x) {
  if (!(x >= -80.0f)) return 0.0f;
  x = fminf(x, 80.0f);
  const float LOG2E = __uint_as_float(0x3FB8AA3Bu);
  const float LN2_HI = __uint_as_float(0x3F317200u);
  const float LN2_LO = __uint_as_float(0x35BFBE8Eu);
  // n = rint(fmul(x, LOG2E)): |x LOG2E| < 2^22, so adding and subtracting 1.5 * 2^23 rounds to the nearest
  // integer, ties to even, exactly as rint does, and leaves n in the low mantissa bits of the sum (both
  // conversions stay off the conversion pipe)
  const float nm = __fadd_rn(__fmul_rn(x, LOG2E), 12582912.0f);
  const float n = __fadd_rn(nm, -12582912.0f);
  float r = __fmaf_rn(n, -LN2_HI, x);
  r = __fmaf_rn(n, -LN2_LO, r);
  float p = __uint_as_float(0x39500D01u);                 // 1/5040
  p = __fmaf_rn(p, r, __uint_as_float(0x3AB60B61u));      // 1/720
  p = __fmaf_rn(p, r, __uint_as_float(0x3C088889u));      // 1/120
  p = __fmaf_rn(p, r, __uint_as_float(0x3D2AAAABu));      // 1/24
  p = __fmaf_rn(p, r, __uint_as_float(0x3E2AAAABu));      // 1/6
  p = __fmaf_rn(p, r, 0.5f);
  p = __fmaf_rn(p, r, 1.0f);
  p = __fmaf_rn(p, r, 1.0f);
  return __uint_as_float(__float_as_uint(p) + (__float_as_uint(nm) << 23));   // bits(nm) = 0x4B400000 + n: the shift keeps n
}

// ---- conversions that stay off the quarter-rate conversion pipe (all exact)
constexpr float kMagicIn = 12583040.0f;   // 1.5 * 2^23 + 128
constexpr float kMagicOut = 12582912.0f;  // 1.5 * 2^23
// int8 byte k of w_xor (= word ^ 0x80808080) as a float: the byte + 128 is placed in the mantissa
// of 1.5 * 2^23 and the offset subtracted
__device__ __forceinline__ float s8_to_f32(uint32_t w_xor, int k) {
  return __fadd_rn(__uint_as_float(__byte_perm(w_xor, 0x4B400000u, 0x7650u + k)), -kMagicIn);
}
// int32 with |v| < 2^22 as a float
__device__ __forceinline__ float i22_to_f32(int v) {
  return __fadd_rn(__int_as_float(v + 0x4B400000), -kMagicOut);
}
// bits whose low byte is the int8 code rne(v) saturated to [-127, 127]: clamping before rounding
// equals rounding before clamping, and (v + 1.5 * 2^23) rounds to nearest even.  The clamp is one
// instruction: min(|v|, 127) with the sign of v put back.  (Used on products of finite factors; a NaN
// would give +-127.)
__device__ __forceinline__ uint32_t rne_clamp_bits(float v) {
  float c;
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c) : "f"(v), "f"(127.0f));
  return __float_as_uint(__fadd_rn(c, kMagicOut));
}
// the same for a pair (the magic addition as one packed instruction)
__device__ __forceinline__ uint2 rne_clamp_bits2(float2 v) {
  float2 c;
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c.x) : "f"(v.x), "f"(127.0f));
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c.y) : "f"(v.y), "f"(127.0f));
  const float2 r = __fadd2_rn(c, make_float2(kMagicOut, kMagicOut));
  return make_uint2(__float_as_uint(r.x), __float_as_uint(r.y));
}
__device__ __forceinline__ uint32_t pack4_bits(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  return __byte_perm(__byte_perm(a, b, 0x0040u), __byte_perm(c, d, 0x0040u), 0x5410u);
}

// Eq. 1 codes without a division per element.  With rcp = frcp_rn(alpha), t = fmul(v, rcp) and
// d = fdiv_rn(v, alpha) differ by at most 1.5 * 2^-23 |v / alpha| < 2.3e-5 wherever the code is not
// saturated, so rne(t) = rne(d) unless t lies that close to a rounding boundary k + 1/2 (ties
// included).  Those elements (about one in 10^4) take the division, and so does every element of a
// step size whose reciprocal may not be a normal number, so the code always equals
// rne(fdiv_rn(v, alpha)) saturated.  quant_code_bits returns bits whose low byte is the code.
struct QuantStep {
  float alpha, rcp, thr;
};
__device__ __forceinline__ QuantStep quant_step(float alpha) {
  QuantStep s;
  s.alpha = alpha;
  s.rcp = __frcp_rn(alpha);
  s.thr = (alpha >= 1e-30f && alpha <= 1e30f) ? 0.49994f : -1.0f;
  return s;
}
__device__ __forceinline__ uint32_t quant_code_bits(float v, const QuantStep& s) {
  const float tc = fminf(fmaxf(__fmul_rn(v, s.rcp), -127.0f), 127.0f);
  const float m = __fadd_rn(tc, kMagicOut);
  const float e = __fsub_rn(tc, __fsub_rn(m, kMagicOut));
  if (fabsf(e) > s.thr) return rne_clamp_bits(__fdiv_rn(v, s.alpha));
  return __float_as_uint(m);
}
// Four codes as one word.  The common path is packed arithmetic and one branch for the four elements:
// products, clamp (min(|t|, 127) with the sign of t), the magic addition, the rounded value and the distance
// of the product from it; only a word with an element near a rounding boundary (or an abnormal step size)
// goes through the divisions, element by element.
__device__ __forceinline__ uint32_t quant_code4(const float4& v, const QuantStep& a, const QuantStep& b,
                                                const QuantStep& c, const QuantStep& d) {
  const float2 t01 = __fmul2_rn(make_float2(v.x, v.y), make_float2(a.rcp, b.rcp));
  const float2 t23 = __fmul2_rn(make_float2(v.z, v.w), make_float2(c.rcp, d.rcp));
  float2 c01, c23;
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c01.x) : "f"(t01.x), "f"(127.0f));
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c01.y) : "f"(t01.y), "f"(127.0f));
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c23.x) : "f"(t23.x), "f"(127.0f));
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c23.y) : "f"(t23.y), "f"(127.0f));
  const float2 mg = make_float2(kMagicOut, kMagicOut), ng = make_float2(-kMagicOut, -kMagicOut);
  const float2 m01 = __fadd2_rn(c01, mg), m23 = __fadd2_rn(c23, mg);
  const float2 m1 = make_float2(-1.0f, -1.0f);   // e = c - (m - magic): both differences are exact
  const float2 e01 = __ffma2_rn(__fadd2_rn(m01, ng), m1, c01), e23 = __ffma2_rn(__fadd2_rn(m23, ng), m1, c23);
  uint32_t b0 = __float_as_uint(m01.x), b1 = __float_as_uint(m01.y), b2 = __float_as_uint(m23.x), b3 = __float_as_uint(m23.y);
  if (fabsf(e01.x) > a.thr || fabsf(e01.y) > b.thr || fabsf(e23.x) > c.thr || fabsf(e23.y) > d.thr) {
    if (fabsf(e01.x) > a.thr) b0 = rne_clamp_bits(__fdiv_rn(v.x, a.alpha));
    if (fabsf(e01.y) > b.thr) b1 = rne_clamp_bits(__fdiv_rn(v.y, b.alpha));
    if (fabsf(e23.x) > c.thr) b2 = rne_clamp_bits(__fdiv_rn(v.z, c.alpha));
    if (fabsf(e23.y) > d.thr) b3 = rne_clamp_bits(__fdiv_rn(v.w, d.alpha));
  }
  return pack4_bits(b0, b1, b2, b3);
}

__device__ __forceinline__ uint32_t pack4(int a, int b, int c, int d) {
  return (uint32_t)(a & 0xff) | ((uint32_t)(b & 0xff) << 8) | ((uint32_t)(c & 0xff) << 16) |
         ((uint32_t)(d & 0xff) << 24);
}

__device__ __forceinline__ int sx8(uint32_t w, int k) { return (int)(int8_t)((w >> (8 * k)) & 0xff); }

// softplus of the raw time step (Algorithm 2 module 1) in binary64, every operation a single correctly
// rounded add, multiply, divide or fused multiply-add in the order written in ssdi8.h, so that the
// binary32 result is defined bit for bit: v = (double)fadd(dt_raw, bias); u = exp(-|v|) by Cody-Waite
// reduction and a degree-13 Taylor polynomial; log(1 + u) = 2 atanh(u / (2 + u)) by its odd series up
// to the 27th power; dt = (float)(max(v, 0) + log(1 + u)).
__device__ __forceinline__ float softplus_dt(float dt_raw, float bias) {
  const double v = (double)__fadd_rn(dt_raw, bias);
  const double a = fabs(v);
  double u = 0.0;
  if (a <= 700.0) {
    const double LOG2E = 0x1.71547652b82fep+0, LN2_HI = 0x1.62e42fee00000p-1, LN2_LO = 0x1.a39ef35793c76p-33;
    const double n = rint(__dmul_rn(-a, LOG2E));
    double r = __fma_rn(n, -LN2_HI, -a);
    r = __fma_rn(n, -LN2_LO, r);
    double p = 1.0 / 6227020800.0;
    p = __fma_rn(p, r, 1.0 / 479001600.0);
    p = __fma_rn(p, r, 1.0 / 39916800.0);
    p = __fma_rn(p, r, 1.0 / 3628800.0);
    p = __fma_rn(p, r, 1.0 / 362880.0);
    p = __fma_rn(p, r, 1.0 / 40320.0);
    p = __fma_rn(p, r, 1.0 / 5040.0);
    p = __fma_rn(p, r, 1.0 / 720.0);
    p = __fma_rn(p, r, 1.0 / 120.0);
    p = __fma_rn(p, r, 1.0 / 24.0);
    p = __fma_rn(p, r, 1.0 / 6.0);
    p = __fma_rn(p, r, 0.5);
    p = __fma_rn(p, r, 1.0);
    p = __fma_rn(p, r, 1.0);
    u = __longlong_as_double(__double_as_longlong(p) + ((long long)__double2int_rn(n) << 52));
  }
  const double s = __ddiv_rn(u, __dadd_rn(2.0, u)), z = __dmul_rn(s, s);
  double q = 1.0 / 27.0;
#pragma unroll
  for (int k = 12; k >= 0; --k) q = __fma_rn(q, z, 1.0 / (double)(2 * k + 1));
  const double lp = __dmul_rn(__dmul_rn(2.0, s), q);
  return (float)__dadd_rn(v > 0.0 ? v : 0.0, lp);
}

// Programmatic dependent launch.  Every kernel of the layer lets its successor in the stream be
// scheduled early (launch_dependents at its start) and itself waits for its predecessor's completion
// and memory flush (pdl_wait) before its first access to global memory, so only work that touches no
// global memory (barrier and tensor-memory set-up, descriptor prefetch) runs under the predecessor's
// tail.  Both are no-ops in a kernel that was launched without the attribute.
// A store whose line is to stay in L2 ahead of ordinary ones (for data a later kernel of the same layer reads
// after other kernels have streamed more than an L2 of traffic in between).
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void st_global_hint(float* a, float v, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(a), "f"(v), "l"(pol) : "memory");
}

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

struct Dims {
  int b, L, H, P, N, G, Q, c;
};

inline Dims make_dims(const ssdi8_dims_t* d) {
  Dims r;
  r.b = d->batch; r.L = d->seqlen; r.H = d->nheads; r.P = d->headdim; r.N = d->dstate;
  r.G = d->ngroups; r.Q = d->chunk; r.c = d->chunk > 0 ? d->seqlen / d->chunk : 0;
  return r;
}

#define SSDI8_CUDA_CHECK(expr)                         \
  do {                                                 \
    cudaError_t e__ = (expr);                          \
    if (e__ != cudaSuccess) return SSDI8_ERR_CUDA;     \
  } while (0)

#define SSDI8_LAUNCH_CHECK()                                       \
  do {                                                             \
    if (cudaPeekAtLastError() != cudaSuccess) {                    \
      (void)cudaGetLastError();                                    \
      return SSDI8_ERR_CUDA;                                       \
    }                                                              \
  } while (0)

}  // namespace ssdi8

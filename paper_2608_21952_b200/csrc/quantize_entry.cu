// Entry quantiser of the SSD layer: the convolution output of a Mamba-2 block is one tensor
// xBC [T][D + 2 G N] (x, then B, then C along the last axis).  One pass reads it (fp32, fp16 or
// bf16) and writes the three int8 tensors the layer consumes, with static step sizes: x per
// channel, B and C per group (quantised once on the group axis at layer entry, before any
// broadcast to heads; Section 4.2 "Quantization of B,C"; Eq. 1 for every element:
// q = rne(fdiv(float(v), alpha)) saturated).  HBM-bound: a thread owns four consecutive columns
// of the concatenated row and walks a slab of rows with several loads in flight.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "kernels.h"

namespace ssdi8 {
namespace {

constexpr int EROWS = 8;

template <typename T> struct Vec4;
template <> struct Vec4<float> {
  typedef float4 raw;
  static __device__ __forceinline__ float4 cvt(const float4& v) { return v; }
};
template <> struct Vec4<__half> {
  typedef uint2 raw;
  static __device__ __forceinline__ float4 cvt(const uint2& v) {
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
    return make_float4(a.x, a.y, b.x, b.y);
  }
};
template <> struct Vec4<__nv_bfloat16> {
  typedef uint2 raw;
  static __device__ __forceinline__ float4 cvt(const uint2& v) {
    // bf16 -> fp32 is a 16-bit shift (exact)
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u),
                       __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
  }
};

template <typename T>
__global__ void __launch_bounds__(128) quant_entry_kernel(const typename Vec4<T>::raw* __restrict__ in,
                                                          const float* __restrict__ s_x,
                                                          const float* __restrict__ s_B,
                                                          const float* __restrict__ s_C,
                                                          uint32_t* __restrict__ xq, uint32_t* __restrict__ Bq,
                                                          uint32_t* __restrict__ Cq, i64 T_, int D, int GN, int N,
                                                          int rows_per_block) {
  const int W4 = (D + 2 * GN) / 4;
  const int q = blockIdx.x * 128 + threadIdx.x;
  if (q >= W4) return;
  const int col = 4 * q;
  float4 s;
  uint32_t* out;
  int ow4, oq;  // output row width and position, in 4-byte words
  if (col < D) {
    s = *reinterpret_cast<const float4*>(s_x + col);
    out = xq; ow4 = D / 4; oq = q;
  } else if (col < D + GN) {
    const float a = s_B[(col - D) / N];
    s = make_float4(a, a, a, a);
    out = Bq; ow4 = GN / 4; oq = (col - D) / 4;
  } else {
    const float a = s_C[(col - D - GN) / N];
    s = make_float4(a, a, a, a);
    out = Cq; ow4 = GN / 4; oq = (col - D - GN) / 4;
  }
  const QuantStep sx = quant_step(s.x), sy = quant_step(s.y), sz = quant_step(s.z), sw = quant_step(s.w);
  const i64 r0 = (i64)blockIdx.y * rows_per_block;
  const i64 r1 = r0 + rows_per_block < T_ ? r0 + rows_per_block : T_;
  i64 r = r0;
  for (; r + EROWS <= r1; r += EROWS) {
    typename Vec4<T>::raw v[EROWS];
#pragma unroll
    for (int u = 0; u < EROWS; ++u) v[u] = __ldcs(in + (r + u) * W4 + q);
#pragma unroll
    for (int u = 0; u < EROWS; ++u) {
      const float4 f = Vec4<T>::cvt(v[u]);
      __stcs(out + (r + u) * ow4 + oq, quant_code4(f, sx, sy, sz, sw));
    }
  }
  for (; r < r1; ++r) {
    const float4 f = Vec4<T>::cvt(__ldcs(in + r * W4 + q));
    __stcs(out + r * ow4 + oq, quant_code4(f, sx, sy, sz, sw));
  }
}

}  // namespace

ssdi8_status_t launch_quantize_entry(const void* xBC, int dtype, i64 T_, int D, int G, int N, const float* s_x,
                                     const float* s_B, const float* s_C, int8_t* xq, int8_t* Bq, int8_t* Cq,
                                     cudaStream_t st) {
  if (T_ == 0) return SSDI8_OK;
  const int GN = G * N, W4 = (D + 2 * GN) / 4;
  const int gx = (W4 + 127) / 128;
  i64 want = (148 * 32 + gx - 1) / gx;
  i64 rows = (T_ + want - 1) / want;
  if (rows < 32) rows = 32;
  rows = (rows + EROWS - 1) / EROWS * EROWS;
  dim3 grid(gx, (unsigned)((T_ + rows - 1) / rows));
  auto X = reinterpret_cast<uint32_t*>(xq);
  auto Bo = reinterpret_cast<uint32_t*>(Bq);
  auto Co = reinterpret_cast<uint32_t*>(Cq);
  if (dtype == 0)
    quant_entry_kernel<float><<<grid, 128, 0, st>>>(static_cast<const float4*>(xBC), s_x, s_B, s_C, X, Bo, Co, T_, D,
                                                    GN, N, (int)rows);
  else if (dtype == 1)
    quant_entry_kernel<__half><<<grid, 128, 0, st>>>(static_cast<const uint2*>(xBC), s_x, s_B, s_C, X, Bo, Co, T_, D,
                                                     GN, N, (int)rows);
  else
    quant_entry_kernel<__nv_bfloat16><<<grid, 128, 0, st>>>(static_cast<const uint2*>(xBC), s_x, s_B, s_C, X, Bo, Co,
                                                            T_, D, GN, N, (int)rows);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

// ChunkCumsum (Algorithm 2, module 1): cs[b,h,k,i] = (float) sum_{i'<=i} (double)dt (double)A_h
// in token order within chunk k, and Gamma[b,h,k] = exp32(cs[.., Q-1]) (Decay_pass, Eq. 5).
// The sum order is part of the definition (it decides rounding downstream), so each
// (b, chunk, head) is scanned sequentially by one thread; loads and stores go through a
// shared-memory tile so that both the [b,L,H] reads and the [b,H,c,Q] writes coalesce.
#include "kernels.h"

namespace ssdi8 {
namespace {

constexpr int CH = 32;  // heads per block

__global__ void __launch_bounds__(256) cumsum_kernel(const float* __restrict__ dt,
                                                     const float* __restrict__ A,
                                                     float* __restrict__ cs,
                                                     float* __restrict__ gamma, Dims d) {
  extern __shared__ float tile[];  // [CH][Q+1]
  const int Q = d.Q, ld = Q + 1;
  const int h0 = blockIdx.x * CH, k = blockIdx.y, b = blockIdx.z;
  const int nh = min(CH, d.H - h0);
  const i64 t0 = (i64)b * d.L + (i64)k * Q;
  for (int e = threadIdx.x; e < Q * CH; e += blockDim.x) {
    int i = e / CH, hh = e % CH;
    if (hh < nh) tile[hh * ld + i] = dt[(t0 + i) * d.H + h0 + hh];
  }
  __syncthreads();
  if (threadIdx.x < nh) {
    const int hh = threadIdx.x;
    const double a = (double)A[h0 + hh];
    double acc = 0.0;
    float last = 0.f;
    for (int i = 0; i < Q; ++i) {
      acc += (double)tile[hh * ld + i] * a;
      last = (float)acc;
      tile[hh * ld + i] = last;
    }
    gamma[((i64)b * d.H + h0 + hh) * d.c + k] = exp32(last);
  }
  __syncthreads();
  for (int e = threadIdx.x; e < Q * CH; e += blockDim.x) {
    int hh = e / Q, i = e % Q;
    if (hh < nh) cs[(((i64)b * d.H + h0 + hh) * d.c + k) * Q + i] = tile[hh * ld + i];
  }
}

}  // namespace

ssdi8_status_t launch_cumsum(const Dims& d, const float* dt, const float* A, float* cs,
                             float* gamma, cudaStream_t st) {
  dim3 grid((d.H + CH - 1) / CH, d.c, d.b);
  size_t smem = sizeof(float) * CH * (d.Q + 1);
  cumsum_kernel<<<grid, 256, smem, st>>>(dt, A, cs, gamma, d);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

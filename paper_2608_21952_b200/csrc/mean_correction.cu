// Estimation of the per-channel mean-correction vector (Eq. 8): the least-squares optimal
// correction of a quantised output is the channel-wise mean of its error,
//   c[ch] = eta * (1 / R) * sum_r (Y[r][ch] - Yq[r][ch]).
// HBM-bound reduction over rows.  Deterministic: each thread owns four channels and sums a slab
// of rows in row order in fp64; a second kernel adds the slab partials in slab order.  No
// floating-point atomics.
#include "kernels.h"

namespace ssdi8 {
namespace {

__global__ void __launch_bounds__(128) mean_err_partial(const float4* __restrict__ y,
                                                        const float4* __restrict__ yq,
                                                        double* __restrict__ partial, i64 R, int ch4,
                                                        int rows_per_slab) {
  const int q = blockIdx.x * 128 + threadIdx.x;
  if (q >= ch4) return;
  const i64 r0 = (i64)blockIdx.y * rows_per_slab;
  const i64 r1 = r0 + rows_per_slab < R ? r0 + rows_per_slab : R;
  double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
  i64 r = r0;
  for (; r + 4 <= r1; r += 4) {
    float4 a[4], b[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      a[u] = __ldcs(y + (r + u) * ch4 + q);
      b[u] = __ldcs(yq + (r + u) * ch4 + q);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      s0 += (double)a[u].x - (double)b[u].x;
      s1 += (double)a[u].y - (double)b[u].y;
      s2 += (double)a[u].z - (double)b[u].z;
      s3 += (double)a[u].w - (double)b[u].w;
    }
  }
  for (; r < r1; ++r) {
    const float4 a = __ldcs(y + r * ch4 + q), b = __ldcs(yq + r * ch4 + q);
    s0 += (double)a.x - (double)b.x;
    s1 += (double)a.y - (double)b.y;
    s2 += (double)a.z - (double)b.z;
    s3 += (double)a.w - (double)b.w;
  }
  double* p = partial + ((i64)blockIdx.y * ch4 + q) * 4;
  p[0] = s0; p[1] = s1; p[2] = s2; p[3] = s3;
}

__global__ void mean_err_final(const double* __restrict__ partial, float* __restrict__ corr, i64 R, int Ch,
                               int nslab, float eta) {
  const int ch = blockIdx.x * blockDim.x + threadIdx.x;
  if (ch >= Ch) return;
  double s = 0.0;
  for (int k = 0; k < nslab; ++k) s += partial[(i64)k * Ch + ch];
  corr[ch] = (float)((double)eta * s / (double)R);
}

}  // namespace

int mean_correction_slabs(i64 R) {
  i64 n = (R + 63) / 64;  // at least 64 rows per slab
  if (n > kMeanCorrMaxSlabs) n = kMeanCorrMaxSlabs;
  if (n < 1) n = 1;
  return (int)n;
}

ssdi8_status_t launch_mean_correction(const float* y, const float* yq, i64 R, i64 Ch, float eta, float* corr,
                                      double* partial, cudaStream_t st) {
  const int ch4 = (int)(Ch / 4);
  const int nslab = mean_correction_slabs(R);
  const int rows = (int)((R + nslab - 1) / nslab);
  dim3 grid((ch4 + 127) / 128, nslab);
  mean_err_partial<<<grid, 128, 0, st>>>(reinterpret_cast<const float4*>(y), reinterpret_cast<const float4*>(yq),
                                         partial, R, ch4, rows);
  SSDI8_LAUNCH_CHECK();
  mean_err_final<<<(unsigned)((Ch + 255) / 256), 256, 0, st>>>(partial, corr, R, (int)Ch, nslab, eta);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

// ChunkCumsum as a kernel of its own (see cumsum_body.cuh for what it computes); the layer step runs
// the same body inside the quantisers' launch.
#include "cumsum_body.cuh"

namespace ssdi8 {
namespace {

// One chunk per block: 8 sequential scans in the scanning warp.  (Four chunks per block, which fills that
// warp's 32 lanes, was measured and is slower, 0.032 against 0.021 ms at batch 8 x 2048 x 80 heads: the
// kernel is bound by the latency of a block's phases, not by the lanes of the scan, and larger blocks
// leave fewer of them to overlap.)
constexpr int kChunksPerBlock = 1;

template <bool SOFTPLUS, bool PRE>
__global__ void __launch_bounds__(256) cumsum_kernel(const float* __restrict__ dt,
                                                     const float* __restrict__ A,
                                                     float* __restrict__ pack,
                                                     float* __restrict__ gamma,
                                                     float* __restrict__ tap_cs, Dims d,
                                                     const float* __restrict__ dt_bias) {
  extern __shared__ float tile[];
  // The wait comes first: a successor that needs nothing of this kernel (the layer step's quantiser of x, B
  // and C) is launched without a wait of its own at its start, so by the time it may be scheduled everything
  // that precedes this kernel in the stream must have completed.
  pdl_wait();
  pdl_launch_dependents();
  cumsum_body<kChunksPerBlock, SOFTPLUS, PRE>(dt, A, pack, gamma, tap_cs, d, blockIdx.x, blockIdx.y, blockIdx.z, tile, dt_bias);
}

// dt = softplus(dt_raw + dt_bias[h]) alone (for callers that calibrate on the positive time step)
__global__ void softplus_dt_kernel(const float* __restrict__ dt_raw, const float* __restrict__ dt_bias,
                                   float* __restrict__ out, i64 n, int H) {
  pdl_launch_dependents();
  pdl_wait();
  const i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x;
  if (e < n) out[e] = softplus_dt(dt_raw[e], dt_bias ? __ldg(dt_bias + (int)(e % H)) : 0.f);
}

}  // namespace

ssdi8_status_t launch_softplus_dt(const float* dt_raw, const float* dt_bias, float* out, i64 rows, int H,
                                  cudaStream_t st) {
  const i64 n = rows * H;
  if (n == 0) return SSDI8_OK;
  if (launch_pdl(softplus_dt_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, dt_raw, dt_bias, out, n, H) !=
      cudaSuccess)
    return SSDI8_ERR_CUDA;
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

ssdi8_status_t launch_cumsum(const Dims& d, const float* dt, const float* A, float* pack,
                             float* gamma, float* tap_cs, cudaStream_t st, const float* dt_bias, bool softplus) {
  dim3 grid((d.H + kCumsumHeads - 1) / kCumsumHeads, (d.c + kChunksPerBlock - 1) / kChunksPerBlock, d.b);
  // a grid that leaves SMs empty is waited for block by block: the variant with the shorter chain
  int dev = 0, sms = 0;
  SSDI8_CUDA_CHECK(cudaGetDevice(&dev));
  SSDI8_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const bool pre = (long long)grid.x * grid.y * grid.z <= sms;
  const size_t smem = cumsum_smem_bytes(d.Q, kChunksPerBlock, pre);
  auto launch = [&](auto kernel) -> ssdi8_status_t {
    SSDI8_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    return launch_pdl(kernel, grid, dim3(256), smem, st, dt, A, pack, gamma, tap_cs, d, dt_bias) == cudaSuccess
               ? SSDI8_OK : SSDI8_ERR_CUDA;
  };
  const ssdi8_status_t ls = softplus ? (pre ? launch(cumsum_kernel<true, true>) : launch(cumsum_kernel<true, false>))
                                     : (pre ? launch(cumsum_kernel<false, true>) : launch(cumsum_kernel<false, false>));
  if (ls != SSDI8_OK) return ls;
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

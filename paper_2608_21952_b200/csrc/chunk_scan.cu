// ChunkScan1 + ChunkScan2 + output sum (Algorithm 2 modules 5, 6), per (batch, chunk, head)
// and 64-row tile of the chunk:
//   acc_off[i,p]  = sum_n Cq[i,n] hq[p,n]                    (INT8 GEMM with the INT8 state)
//   Mq[i,j]       = per-row re-quantised  CBq[i,j] dt_j exp(cs_i - cs_j), j <= i   (see ssdi8.h)
//   acc_diag[i,p] = sum_j Mq[i,j] xq[j,p]
//   y = exp(cs_i) s_C s_h acc_off + (s_cb rowmax_i / 127) s_x acc_diag + D s_x xq + corr
#include "kernels.h"
#include "mma_s8.cuh"

namespace ssdi8 {
namespace {

constexpr int TM = 64;  // rows per block = sub-block length SB of the decay factorisation

__global__ void __launch_bounds__(128) chunk_scan_kernel(
    const int8_t* __restrict__ xq, const int8_t* __restrict__ Cq, const int8_t* __restrict__ CBq,
    const int8_t* __restrict__ hq, const float* __restrict__ s_x, const float* __restrict__ s_C,
    const float* __restrict__ s_cb, const float* __restrict__ s_h, const float* __restrict__ dt,
    const float* __restrict__ cs, const float* __restrict__ D, const float* __restrict__ corr,
    float* __restrict__ y, ScanTaps taps, Dims d) {
  extern __shared__ __align__(16) int8_t smem[];
  const int Q = d.Q, P = d.P, N = d.N;
  const int ldn = N + 16, ldq = Q + 16;
  const int it = blockIdx.x % (Q / TM), h = blockIdx.x / (Q / TM), k = blockIdx.y, b = blockIdx.z;
  const int g = h / (d.H / d.G);
  const int KJ = (it + 1) * TM;  // causal extent of this row tile
  int8_t* Cs = smem;                       // [TM][ldn]
  int8_t* Hs = Cs + TM * ldn;              // [P][ldn]
  int8_t* Ms = Hs + P * ldn;               // [TM][ldq]
  int8_t* XT = Ms + TM * ldq;              // [P][ldq]   xq transposed: row p, token contiguous
  int8_t* CBs = XT + P * ldq;              // [TM][Q]
  float* cs_s = reinterpret_cast<float*>(CBs + TM * Q);  // [Q]
  float* dt_s = cs_s + Q;                                // [Q]
  float* rm_s = dt_s + Q;                                // [TM]
  const i64 tok0 = (i64)b * d.L + (i64)k * Q;
  const int tid = threadIdx.x;
  const int nw = N / 4;
  for (int e = tid; e < TM * nw; e += blockDim.x) {
    const int r = e / nw, w = e % nw;
    *reinterpret_cast<uint32_t*>(Cs + r * ldn + 4 * w) =
        *reinterpret_cast<const uint32_t*>(Cq + ((tok0 + it * TM + r) * d.G + g) * N + 4 * w);
  }
  const int8_t* hqk = hq + ((((i64)b * d.c + k) * d.H + h) * P) * N;
  for (int e = tid; e < P * nw; e += blockDim.x) {
    const int r = e / nw, w = e % nw;
    *reinterpret_cast<uint32_t*>(Hs + r * ldn + 4 * w) =
        *reinterpret_cast<const uint32_t*>(hqk + r * N + 4 * w);
  }
  const int pw = P / 4;
  for (int e = tid; e < KJ * pw; e += blockDim.x) {
    const int j = e / pw, w4 = e % pw;
    const uint32_t w = *reinterpret_cast<const uint32_t*>(xq + ((tok0 + j) * d.H + h) * P + 4 * w4);
#pragma unroll
    for (int u = 0; u < 4; ++u) XT[(4 * w4 + u) * ldq + j] = (int8_t)sx8(w, u);
  }
  const int8_t* cbk = CBq + (((i64)b * d.c + k) * d.G + g) * Q * Q + (i64)it * TM * Q;
  const int kw = KJ / 4;
  for (int e = tid; e < TM * kw; e += blockDim.x) {
    const int r = e / kw, w = e % kw;
    *reinterpret_cast<uint32_t*>(CBs + r * Q + 4 * w) =
        *reinterpret_cast<const uint32_t*>(cbk + r * Q + 4 * w);
  }
  const float* csk = cs + (((i64)b * d.H + h) * d.c + k) * Q;
  for (int j = tid; j < Q; j += blockDim.x) {
    cs_s[j] = csk[j];
    dt_s[j] = dt[(tok0 + j) * d.H + h];
  }
  __syncthreads();

  // ---- masked operand, two threads per output row (sub-blocks J = s, s+2, ...)
  {
    const int r = tid >> 1, s = tid & 1;
    const int i = it * TM + r, I = it;
    const float cs_i = cs_s[i];
    float rmax = 0.f;
    for (int J = s; J <= I; J += 2) {
      const int je = J * TM + TM - 1;
      const int jend = (J == I) ? i : je;
      const float f = (J == I) ? 1.0f : exp32(__fsub_rn(cs_i, cs_s[je]));
      const float ref = (J == I) ? cs_i : cs_s[je];
      float bmax = 0.f;
      for (int j = J * TM; j <= jend; ++j) {
        const float w = __fmul_rn(dt_s[j], exp32(__fsub_rn(ref, cs_s[j])));
        bmax = fmaxf(bmax, fabsf(__fmul_rn((float)CBs[r * Q + j], w)));
      }
      rmax = fmaxf(rmax, __fmul_rn(bmax, f));
    }
    rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, 1));
    const float inv = (rmax >= 1e-30f) ? __fdiv_rn(127.0f, rmax) : 0.f;
    if (s == 0) {
      rm_s[r] = rmax;
      if (taps.rowmax) taps.rowmax[(tok0 + i) * d.H + h] = rmax;
    }
    int8_t* mq_tap = taps.Mq ? taps.Mq + ((((i64)b * d.c + k) * d.H + h) * Q + i) * Q : nullptr;
    for (int J = s; J <= I; J += 2) {
      const int je = J * TM + TM - 1;
      const int jend = (J == I) ? i : je;
      const float f = (J == I) ? 1.0f : exp32(__fsub_rn(cs_i, cs_s[je]));
      const float ref = (J == I) ? cs_i : cs_s[je];
      const float gf = __fmul_rn(f, inv);
      for (int j = J * TM; j <= je; ++j) {
        int q = 0;
        if (j <= jend) {
          const float w = __fmul_rn(dt_s[j], exp32(__fsub_rn(ref, cs_s[j])));
          q = rne_clamp(__fmul_rn(__fmul_rn((float)CBs[r * Q + j], w), gf));
        }
        Ms[r * ldq + j] = (int8_t)q;
        if (mq_tap) mq_tap[j] = (int8_t)q;
      }
    }
  }
  __syncthreads();

  // ---- the two integer GEMMs: warp w owns rows 16 w .. 16 w + 15, all P columns
  const int warp = tid >> 5, lane = tid & 31;
  int acc_off[8][4], acc_diag[8][4];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int e = 0; e < 4; ++e) { acc_off[a][e] = 0; acc_diag[a][e] = 0; }
  warp_gemm_s8<8>(acc_off, Cs, ldn, warp * 16, Hs, ldn, 0, N);
  warp_gemm_s8<8>(acc_diag, Ms, ldq, warp * 16, XT, ldq, 0, KJ);

  // ---- epilogue
  const float sC = s_C[g], scb = s_cb[g];
  const float Dh = D ? D[h] : 0.f;
#pragma unroll
  for (int e2 = 0; e2 < 2; ++e2) {
    const int r = warp * 16 + (lane >> 2) + 8 * e2;
    const int i = it * TM + r;
    const float dec = exp32(cs_s[i]) * sC;
    const float sm = scb * rm_s[r] * (1.0f / 127.0f);
#pragma unroll
    for (int a = 0; a < 8; ++a) {
      float v[2];
#pragma unroll
      for (int e1 = 0; e1 < 2; ++e1) {
        const int p = 8 * a + 2 * (lane & 3) + e1;
        const int e = 2 * e2 + e1;
        const float sxp = s_x[h * P + p];
        float t = dec * s_h[h * P + p] * (float)acc_off[a][e] + sm * sxp * (float)acc_diag[a][e];
        t += Dh * sxp * (float)XT[p * ldq + i];
        if (corr) t += corr[h * P + p];
        v[e1] = t;
        const i64 o = ((tok0 + i) * d.H + h) * P + p;
        if (taps.acc_off) taps.acc_off[o] = acc_off[a][e];
        if (taps.acc_diag) taps.acc_diag[o] = acc_diag[a][e];
      }
      const i64 o = ((tok0 + i) * d.H + h) * P + 8 * a + 2 * (lane & 3);
      *reinterpret_cast<float2*>(y + o) = make_float2(v[0], v[1]);
    }
  }
}

}  // namespace

ssdi8_status_t launch_chunk_scan(const Dims& d, const int8_t* xq, const int8_t* Cq,
                                 const int8_t* CBq, const int8_t* hq, const float* s_x,
                                 const float* s_C, const float* s_cb, const float* s_h,
                                 const float* dt, const float* cs, const float* D,
                                 const float* corr, float* y, const ScanTaps& taps,
                                 cudaStream_t st) {
  dim3 grid(d.H * (d.Q / TM), d.c, d.b);
  size_t smem = (size_t)(TM + d.P) * (d.N + 16) + (size_t)(TM + d.P) * (d.Q + 16) +
                (size_t)TM * d.Q + sizeof(float) * (2 * d.Q + TM);
  static bool attr_done = false;
  if (!attr_done) {
    SSDI8_CUDA_CHECK(cudaFuncSetAttribute(chunk_scan_kernel,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
    attr_done = true;
  }
  chunk_scan_kernel<<<grid, 128, smem, st>>>(xq, Cq, CBq, hq, s_x, s_C, s_cb, s_h, dt, cs, D, corr,
                                             y, taps, d);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

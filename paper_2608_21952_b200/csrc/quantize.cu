// Activation quantiser (Eq. 1): uniform symmetric 8-bit with one step size per channel
// of the view in[R][Ch][I].  HBM-bound: 16-byte loads, 4-byte packed stores, every warp
// instruction fully coalesced; absmax by per-thread running maxima, warp shuffles and
// one order-independent atomicMax on the (non-negative) binary32 bit pattern.
#include "kernels.h"

namespace ssdi8 {
namespace {

constexpr int QT = 256;      // threads per block
constexpr int QUNROLL = 4;   // float4 loads in flight per thread

// ---- quantise, I == 1: 4 consecutive elements are 4 consecutive channels.  A thread owns one
// float4 column (its four step sizes stay in registers) and walks a slab of rows with QROWS
// independent 16-byte loads in flight; a warp reads 512 and writes 128 contiguous bytes per row.
constexpr int QROWS = 8;
__global__ void __launch_bounds__(128) quant_ch_fastest(const float4* __restrict__ in,
                                                        const float4* __restrict__ scale,
                                                        uint32_t* __restrict__ out, i64 R, int ch4,
                                                        int rows_per_block) {
  const int q = blockIdx.x * 128 + threadIdx.x;
  if (q >= ch4) return;
  const float4 s = __ldg(scale + q);
  const QuantStep sx = quant_step(s.x), sy = quant_step(s.y), sz = quant_step(s.z), sw = quant_step(s.w);
  const i64 r0 = (i64)blockIdx.y * rows_per_block;
  const i64 r1 = r0 + rows_per_block < R ? r0 + rows_per_block : R;
  i64 r = r0;
  for (; r + QROWS <= r1; r += QROWS) {
    float4 v[QROWS];
#pragma unroll
    for (int u = 0; u < QROWS; ++u) v[u] = __ldcs(in + (r + u) * ch4 + q);
#pragma unroll
    for (int u = 0; u < QROWS; ++u)
      __stcs(out + (r + u) * ch4 + q, quant_code4(v[u], sx, sy, sz, sw));
  }
  for (; r < r1; ++r) {
    const float4 v = __ldcs(in + r * ch4 + q);
    __stcs(out + r * ch4 + q, quant_code4(v, sx, sy, sz, sw));
  }
}

// ---- the layer's three static quantisers (x per channel; B and C per group) as one launch.  Every
// tensor is a matrix of R rows; a block covers up to 128 float4 columns and, where a row is narrower
// than that, several rows per pass, so that a warp still reads 512 contiguous bytes.  The jobs of the
// narrow tensors come first in the grid: they are placed at once and finish under the wide one.
struct QuantJob {
  const float4* in; const float* scale; uint32_t* out;
  int ch4;          // float4 per row
  int tpr;          // threads per row (a power of two <= 128)
  int gx;           // column blocks per row
  int shift;        // step size of channel c = scale[c >> shift]
  int first_block;  // of this job in the grid
  int rows;         // rows per block
};
struct QuantJobs {
  QuantJob job[3]; i64 R;
  int late_wait;   // 1: launched right behind ChunkCumsum of the same layer, which it does not depend on (see the kernel)
};

__global__ void __launch_bounds__(128, 8) quant_jobs(const QuantJobs a) {
  pdl_launch_dependents();
  // Programmatic dependent launch.  Normally: wait for the predecessor before the first global access.
  // Launched right behind ChunkCumsum (which waits for ITS predecessor before it lets this kernel be
  // scheduled, and whose outputs this kernel does not touch), the blocks start at once and work beside
  // that kernel.  The wait moves to the end of the grid's last block (one waiting block is enough, and a
  // wait in every block would keep the early ones resident until ChunkCumsum has finished): it keeps
  // "this kernel complete" implying "ChunkCumsum complete" for the state kernel that follows, and by then
  // it returns at once.
  if (!a.late_wait) pdl_wait();
  struct LateWait {
    bool on;
    __device__ ~LateWait() { if (on) pdl_wait(); }
  } late_wait_at_exit{a.late_wait != 0 && blockIdx.x == gridDim.x - 1};
  const int blk = (int)blockIdx.x;
  const int jb = blk >= a.job[2].first_block ? 2 : blk >= a.job[1].first_block ? 1 : 0;
  const QuantJob& j = a.job[jb];
  const int rel = blk - j.first_block;
  const int bx = rel % j.gx, by = rel / j.gx;
  const int tr = threadIdx.x / j.tpr;          // row of this thread within a pass
  const int rpp = 128 / j.tpr;                 // rows per pass
  const int q = bx * j.tpr + (threadIdx.x & (j.tpr - 1));
  if (q >= j.ch4) return;
  float4 s;
  if (j.shift == 0) {
    s = __ldg(reinterpret_cast<const float4*>(j.scale) + q);
  } else {
    const float g = __ldg(j.scale + ((q * 4) >> j.shift));   // 4 consecutive channels share a group
    s = make_float4(g, g, g, g);
  }
  const QuantStep sx = quant_step(s.x), sy = quant_step(s.y), sz = quant_step(s.z), sw = quant_step(s.w);
  const i64 r0 = (i64)by * j.rows + tr;
  const i64 r1 = (i64)(by + 1) * j.rows < a.R ? (i64)(by + 1) * j.rows : a.R;
  if (r0 >= r1) return;
  // (the launcher keeps every tensor below 2^31 float4, so 32-bit element indices do)
  const uint32_t stride = (uint32_t)(rpp * j.ch4);   // float4 (and code words) between two passes
  uint32_t e = (uint32_t)r0 * (uint32_t)j.ch4 + (uint32_t)q;
  int left = (int)((r1 - r0 + rpp - 1) / rpp);       // passes this thread takes
  const float4* __restrict__ in = j.in;
  uint32_t* __restrict__ out = j.out;
  for (; left >= QROWS; left -= QROWS, e += QROWS * stride) {
    float4 v[QROWS];
#pragma unroll
    for (int u = 0; u < QROWS; ++u) v[u] = __ldcs(in + (e + u * stride));
#pragma unroll
    for (int u = 0; u < QROWS; ++u) out[e + u * stride] = quant_code4(v[u], sx, sy, sz, sw);
  }
  for (; left > 0; --left, e += stride) out[e] = quant_code4(__ldcs(in + e), sx, sy, sz, sw);
}

// ---- quantise, I % 4 == 0: 4 consecutive elements share a channel
__global__ void __launch_bounds__(QT) quant_inner(const float4* __restrict__ in,
                                                  const float* __restrict__ scale,
                                                  uint32_t* __restrict__ out, uint32_t n4,
                                                  uint32_t I4, uint32_t Ch) {
  uint32_t base = blockIdx.x * (QT * QUNROLL) + threadIdx.x;
#pragma unroll
  for (int u = 0; u < QUNROLL; ++u) {
    uint32_t e = base + u * QT;
    if (e < n4) {
      float4 v = __ldcs(in + e);
      const QuantStep s = quant_step(__ldg(scale + (e / I4) % Ch));
      out[e] = quant_code4(v, s, s, s, s);
    }
  }
}

// ---- absmax, I == 1.  Thread owns 4 channels and walks rows; grid.y splits the rows.
__global__ void __launch_bounds__(QT) absmax_ch_fastest(const float4* __restrict__ in,
                                                        uint32_t* __restrict__ bits, i64 R, int ch4,
                                                        int rows_per_block) {
  int q = blockIdx.x * QT + threadIdx.x;
  if (q >= ch4) return;
  i64 r0 = (i64)blockIdx.y * rows_per_block;
  i64 r1 = r0 + rows_per_block < R ? r0 + rows_per_block : R;
  float4 m = make_float4(0.f, 0.f, 0.f, 0.f);
  i64 r = r0;
  for (; r + 4 <= r1; r += 4) {
    float4 v0 = __ldg(in + (r + 0) * ch4 + q), v1 = __ldg(in + (r + 1) * ch4 + q);
    float4 v2 = __ldg(in + (r + 2) * ch4 + q), v3 = __ldg(in + (r + 3) * ch4 + q);
    m.x = fmaxf(fmaxf(fmaxf(m.x, fabsf(v0.x)), fmaxf(fabsf(v1.x), fabsf(v2.x))), fabsf(v3.x));
    m.y = fmaxf(fmaxf(fmaxf(m.y, fabsf(v0.y)), fmaxf(fabsf(v1.y), fabsf(v2.y))), fabsf(v3.y));
    m.z = fmaxf(fmaxf(fmaxf(m.z, fabsf(v0.z)), fmaxf(fabsf(v1.z), fabsf(v2.z))), fabsf(v3.z));
    m.w = fmaxf(fmaxf(fmaxf(m.w, fabsf(v0.w)), fmaxf(fabsf(v1.w), fabsf(v2.w))), fabsf(v3.w));
  }
  for (; r < r1; ++r) {
    float4 v = __ldg(in + r * ch4 + q);
    m.x = fmaxf(m.x, fabsf(v.x)); m.y = fmaxf(m.y, fabsf(v.y));
    m.z = fmaxf(m.z, fabsf(v.z)); m.w = fmaxf(m.w, fabsf(v.w));
  }
  // step size of this partial maximum: fdiv by a positive constant is monotone, so the
  // maximum of the step sizes is the step size of the maximum
  atomicMax(bits + 4 * q + 0, __float_as_uint(__fdiv_rn(m.x, 127.0f)));
  atomicMax(bits + 4 * q + 1, __float_as_uint(__fdiv_rn(m.y, 127.0f)));
  atomicMax(bits + 4 * q + 2, __float_as_uint(__fdiv_rn(m.z, 127.0f)));
  atomicMax(bits + 4 * q + 3, __float_as_uint(__fdiv_rn(m.w, 127.0f)));
}

// ---- absmax, I % 4 == 0.  Block (x = row split, y = channel) reduces its rows of one channel.
__global__ void __launch_bounds__(QT) absmax_inner(const float4* __restrict__ in,
                                                   uint32_t* __restrict__ bits, i64 R, int Ch, int I4,
                                                   int rows_per_block) {
  __shared__ float red[QT / 32];
  int ch = blockIdx.y;
  i64 r0 = (i64)blockIdx.x * rows_per_block;
  i64 r1 = r0 + rows_per_block < R ? r0 + rows_per_block : R;
  i64 cnt = (r1 - r0) * I4;
  float m = 0.f;
  for (i64 e = threadIdx.x; e < cnt; e += QT) {
    i64 r = r0 + e / I4;
    int i = (int)(e % I4);
    float4 v = __ldg(in + (r * Ch + ch) * I4 + i);
    m = fmaxf(fmaxf(fmaxf(m, fabsf(v.x)), fmaxf(fabsf(v.y), fabsf(v.z))), fabsf(v.w));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 1; w < QT / 32; ++w) m = fmaxf(m, red[w]);
    atomicMax(bits + ch, __float_as_uint(__fdiv_rn(m, 127.0f)));
  }
}

__global__ void finalize_alpha(uint32_t* bits, i64 n) {
  i64 k = (i64)blockIdx.x * blockDim.x + threadIdx.x;
  if (k < n && bits[k] == 0u) bits[k] = __float_as_uint(1.0f);  // all-zero channel: alpha = 1
}

}  // namespace

ssdi8_status_t launch_quantize(const float* in, i64 R, i64 Ch, i64 I, float* scale, int mode,
                               int8_t* out, cudaStream_t st) {
  const i64 n4 = R * Ch * I / 4;
  if (n4 == 0) return SSDI8_OK;
  uint32_t* bits = reinterpret_cast<uint32_t*>(scale);
  if (mode == 1 || mode == 2) {
    if (mode == 1) SSDI8_CUDA_CHECK(cudaMemsetAsync(scale, 0, sizeof(float) * Ch, st));
    if (I == 1) {
      int ch4 = (int)(Ch / 4);
      int gx = (ch4 + QT - 1) / QT;
      // enough row splits to fill the machine, at least 64 rows each
      i64 want = (148 * 8 + gx - 1) / gx;
      i64 rows = (R + want - 1) / want;
      if (rows < 64) rows = 64;
      int gy = (int)((R + rows - 1) / rows);
      absmax_ch_fastest<<<dim3(gx, gy), QT, 0, st>>>(reinterpret_cast<const float4*>(in), bits, R,
                                                      ch4, (int)rows);
    } else {
      int I4 = (int)(I / 4);
      i64 want = (148 * 8 + Ch - 1) / Ch;
      i64 rows = (R + want - 1) / want;
      i64 min_rows = (QT * 4 + I4 - 1) / I4;
      if (rows < min_rows) rows = min_rows;
      int gx = (int)((R + rows - 1) / rows);
      absmax_inner<<<dim3(gx, (unsigned)Ch), QT, 0, st>>>(reinterpret_cast<const float4*>(in), bits,
                                                           R, (int)Ch, I4, (int)rows);
    }
    SSDI8_LAUNCH_CHECK();
    if (mode == 1) {
      finalize_alpha<<<(unsigned)((Ch + 255) / 256), 256, 0, st>>>(bits, Ch);
      SSDI8_LAUNCH_CHECK();
    }
  }
  if (!out) return SSDI8_OK;
  unsigned grid = (unsigned)((n4 + QT * QUNROLL - 1) / (QT * QUNROLL));
  if (I == 1) {
    const int ch4 = (int)(Ch / 4);
    const int gx = (ch4 + 127) / 128;
    // slabs of rows: enough blocks to fill the machine several times over, at least 32 rows each
    i64 want = (148 * 32 + gx - 1) / gx;
    i64 rows = (R + want - 1) / want;
    if (rows < 32) rows = 32;
    rows = (rows + QROWS - 1) / QROWS * QROWS;
    const int gy = (int)((R + rows - 1) / rows);
    quant_ch_fastest<<<dim3(gx, gy), 128, 0, st>>>(reinterpret_cast<const float4*>(in),
                                                   reinterpret_cast<const float4*>(scale),
                                                   reinterpret_cast<uint32_t*>(out), R, ch4, (int)rows);
  }
  else
    quant_inner<<<grid, QT, 0, st>>>(reinterpret_cast<const float4*>(in), scale,
                                     reinterpret_cast<uint32_t*>(out), (uint32_t)n4, (uint32_t)(I / 4),
                                     (uint32_t)Ch);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

ssdi8_status_t launch_quantize_xbc(const float* x, const float* B, const float* C, i64 T_, int D, int G, int N,
                                   const float* s_x, const float* s_B, const float* s_C, int8_t* xq, int8_t* Bq,
                                   int8_t* Cq, cudaStream_t st, bool after_cumsum) {
  if (T_ == 0) return SSDI8_OK;
  if (T_ * D / 4 >= ((i64)1 << 31) || T_ * G * N / 4 >= ((i64)1 << 31)) return SSDI8_ERR_UNSUPPORTED;
  QuantJobs a;
  a.R = T_;
  int shift = 0;
  while ((1 << shift) < N) ++shift;   // N is a power of two here (the caller checks)
  auto fill = [&](QuantJob& j, const float* in, const float* sc, int8_t* out, int width, int sh, int first) {
    j.in = reinterpret_cast<const float4*>(in);
    j.scale = sc;
    j.out = reinterpret_cast<uint32_t*>(out);
    j.ch4 = width / 4;
    j.tpr = 128;
    while (j.tpr / 2 >= j.ch4 && j.tpr > 1) j.tpr /= 2;
    j.gx = (j.ch4 + j.tpr - 1) / j.tpr;
    j.shift = sh;
    j.first_block = first;
    // short slabs: blocks that live a few microseconds each, so that a kernel running beside this one finds
    // free slots all the time (a slab is at least one full round of QROWS passes)
    j.rows = QROWS * (128 / j.tpr) < 16 ? 16 : QROWS * (128 / j.tpr);
    return first + j.gx * (int)((T_ + j.rows - 1) / j.rows);
  };
  int nb = fill(a.job[0], B, s_B, Bq, G * N, shift, 0);
  nb = fill(a.job[1], C, s_C, Cq, G * N, shift, nb);
  nb = fill(a.job[2], x, s_x, xq, D, 0, nb);
  a.late_wait = after_cumsum ? 1 : 0;
  if (launch_pdl(quant_jobs, dim3((unsigned)nb), dim3(128), 0, st, a) != cudaSuccess) return SSDI8_ERR_CUDA;
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

// bits[k] holds either a binary32 absmax or (bits_are_int) an int32 absmax; the step size is
// fdiv(fmul(value, fmul(mul_a[k], mul_b[k])), 127) (multipliers optional), 1 if the value is 0.
namespace {
__global__ void finalize_scales_k(float* s, i64 n, const float* mul_a, const float* mul_b,
                                  int bits_are_int) {
  i64 k = (i64)blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= n) return;
  uint32_t u = __float_as_uint(s[k]);
  if (u == 0u) { s[k] = 1.0f; return; }
  float v = bits_are_int ? (float)(int)u : s[k];
  if (mul_a) v = __fmul_rn(v, __fmul_rn(mul_a[k], mul_b[k]));
  s[k] = __fdiv_rn(v, 127.0f);
}
}  // namespace

ssdi8_status_t launch_finalize_scales(float* scale_bits, i64 n, const float* mul_a,
                                      const float* mul_b, int bits_are_int, cudaStream_t st) {
  finalize_scales_k<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(scale_bits, n, mul_a, mul_b,
                                                                 bits_are_int);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

// ChunkScan1 + ChunkScan2 + output sum (Algorithm 2 modules 5, 6) on tcgen05 tensor cores.
// One CTA per (batch, chunk, head) and 128-row tile of the chunk:
//   acc_off[i,p]  = sum_n Cq[i,n] hq[p,n]                 INT8 MMA, INT32 accumulator in TMEM
//   Mq[i,j]       = per-row re-quantised CBq[i,j] dt_j exp(cs_i - cs_j), j <= i   (see ssdi8.h)
//   acc_diag[i,p] = sum_j Mq[i,j] xq[j,p]                 INT8 MMA, second TMEM accumulator
//   y = exp(cs_i) s_C s_h acc_off + (s_cb rowmax_i / 127) s_x acc_diag + D s_x xq + corr
// Operand tiles are staged by TMA in the swizzled layouts the MMA reads (Cq, hq, CBq K-major,
// xq MN-major); Mq is written in place over CBq; y leaves through a swizzled staging tile and
// two TMA stores.  No multicast, one CTA per tile, every wait is bounded.
#include "kernels.h"
#include "sm100.cuh"

namespace ssdi8 {
namespace {

using namespace sm100;

struct ScanArgs {
  const float* s_x; const float* s_C; const float* s_cb; const float* s_h;
  const float* dt; const float* cs; const float* D; const float* corr;
  int32_t* status;
  ScanTaps taps;
  Dims d;
};

constexpr int kThreads = 256;
constexpr uint32_t kTmemCols = 128;  // acc_off: columns 0..63, acc_diag: columns 64..127
// shared-memory carve-up (bytes, from a 1024-byte aligned base)
constexpr uint32_t OFF_C = 0;             // [128][N]        Cq tile, K-major
constexpr uint32_t OFF_H = 16384;         // [64][N]         hq tile, K-major
constexpr uint32_t OFF_X = 24576;         // [256][64]       xq rows, MN-major
constexpr uint32_t OFF_CB = 40960;        // 2 x [128][128]  CBq panels -> Mq in place -> y staging
constexpr uint32_t OFF_F = 73728;         // float arrays
constexpr uint32_t SMEM_BYTES = OFF_F + 5 * 256 * 4 + 3 * 64 * 4 + 64;
constexpr uint32_t PANEL = 16384;

__device__ __forceinline__ float unpack_s8(uint32_t w_xor, int k) {
  // w_xor = word ^ 0x80808080: byte + 128 goes into the mantissa of 1.5 * 2^23
  return __fadd_rn(__uint_as_float(__byte_perm(w_xor, 0x4B400000u, 0x7650u + k)), -12583040.0f);
}
// rne(v) for |v| < 2^22 sits in the low bits of (v + 1.5 * 2^23); callers guarantee |v| < 127.5
__device__ __forceinline__ uint32_t rne_bits(float v) { return __float_as_uint(__fadd_rn(v, 12582912.0f)); }
__device__ __forceinline__ uint32_t pack4_bits(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  return __byte_perm(__byte_perm(a, b, 0x0040u), __byte_perm(c, d, 0x0040u), 0x5410u);
}

__global__ void __launch_bounds__(kThreads, 2)
chunk_scan_tc(const __grid_constant__ CUtensorMap tm_C, const __grid_constant__ CUtensorMap tm_h,
              const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_cb,
              const __grid_constant__ CUtensorMap tm_y, const ScanArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const Dims& d = a.d;
  const int Q = d.Q, N = d.N, P = d.P;
  const int TM = Q < 128 ? Q : 128;        // valid rows of a tile
  const int ntile = Q / TM;
  const uint32_t RBN = N, RBQ = TM;        // row bytes of the N-contracted and Q-contracted tiles
  const int it = blockIdx.x % ntile;
  int u = blockIdx.x / ntile;
  const int h = u % d.H; u /= d.H;
  const int k = u % d.c;
  const int b = u / d.c;
  const int g = h / (d.H / d.G);
  const int KJ = (it + 1) * TM;            // causal extent of this row tile
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const i64 tok0 = (i64)b * d.L + (i64)k * Q;

  uint8_t* sC = smem + OFF_C;
  uint8_t* sH = smem + OFF_H;
  uint8_t* sX = smem + OFF_X;
  uint8_t* sCB = smem + OFF_CB;
  float* cs_s = reinterpret_cast<float*>(smem + OFF_F);
  float* dt_s = cs_s + 256;
  float* woff_s = dt_s + 256;
  float* part_s = woff_s + 256;
  float* atok_s = part_s + 256;  // per-token decay a_m = exp32(cs_m - cs_{m-1})
  float* colA = atok_s + 256;  // s_C s_h[p]
  float* colB = colA + 64;     // s_x[p]
  float* colC = colB + 64;     // corr[p]
  uint64_t* bars = reinterpret_cast<uint64_t*>(colC + 64);  // [0] C+h, [1] CBq, [2] xq, [3] MMA done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);

  if (tid == 0) {
    for (int i = 0; i < 4; ++i) mbar_init(&bars[i], 1);
    fence_mbar_init();
    tma_prefetch_desc(&tm_C); tma_prefetch_desc(&tm_h); tma_prefetch_desc(&tm_x);
    tma_prefetch_desc(&tm_cb); tma_prefetch_desc(&tm_y);
  }
  if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (tid == 0) {
    mbar_expect_tx(&bars[0], (uint32_t)(TM * N + 64 * N));
    tma_load_3d(sC, &tm_C, &bars[0], 0, g, (int)(tok0 + it * TM));
    tma_load_2d(sH, &tm_h, &bars[0], 0, (int)((((i64)b * d.c + k) * d.H + h) * P));
    const int npanel = KJ / (int)RBQ;
    mbar_expect_tx(&bars[1], (uint32_t)(npanel * TM * RBQ));
    for (int pn = 0; pn < npanel; ++pn)
      tma_load_2d(sCB + pn * PANEL, &tm_cb, &bars[1], pn * (int)RBQ,
                  (int)((((i64)b * d.c + k) * d.G + g) * Q + it * TM));
    mbar_expect_tx(&bars[2], (uint32_t)(KJ * 64));
    for (int j0 = 0; j0 < KJ; j0 += TM) tma_load_3d(sX + j0 * 64, &tm_x, &bars[2], 0, h, (int)(tok0 + j0));
  }

  // ---- per-token and per-column scalars
  const float* csk = a.cs + (((i64)b * d.H + h) * d.c + k) * Q;
  if (tid < Q) {
    cs_s[tid] = csk[tid];
    dt_s[tid] = a.dt[(tok0 + tid) * d.H + h];
  }
  if (tid < 64) {
    colA[tid] = a.s_C[g] * a.s_h[h * P + tid];
    colB[tid] = a.s_x[h * P + tid];
    colC[tid] = a.corr ? a.corr[h * P + tid] : 0.f;
  }
  __syncthreads();
  // weight of column j as seen from a later sub-block: dt_j exp(cs_je - cs_j), je = end of j's sub-block
  if (tid < KJ) {
    woff_s[tid] = __fmul_rn(dt_s[tid], exp32(__fsub_rn(cs_s[tid | 63], cs_s[tid])));
    atok_s[tid] = tid > 0 ? exp32(__fsub_rn(cs_s[tid], cs_s[tid - 1])) : 1.0f;
  }

  // ---- ChunkScan1 MMA: acc_off = Cq * hq^T   (overlaps the mask computation below)
  if (tid == 0) {
    mbar_wait(&bars[0], 0, a.status);
    tc_fence_after();
    const uint32_t idesc = idesc_s8(128, 64, 0, 0);
    for (int s = 0; s < N / 32; ++s)
      mma_s8_ss(tmem, tile_desc(smem_u32(sC) + 32 * s, RBN), tile_desc(smem_u32(sH) + 32 * s, RBN), idesc,
                s > 0);
  }
  __syncthreads();  // woff_s visible

  // ---- masked operand Mq, in place over CBq.  Thread pair per row: role 0 owns the row's own
  // (diagonal) sub-block, role 1 the earlier sub-blocks and the zero fill of later ones.
  const int r = tid & 127, role = tid >> 7;
  const bool row_ok = r < TM;
  const int i = it * TM + r;           // row within the chunk
  const int I = i >> 6;                // its sub-block
  const int nblk = KJ >> 6;            // sub-blocks in the contraction range
  const uint32_t cpp = RBQ >> 4;       // 16-byte chunks per panel row
  auto chunk_ptr = [&](int j16) -> uint4* {  // 16-byte chunk j16 (columns 16 j16 ..) of row r
    const uint32_t pn = (uint32_t)j16 / cpp, c = (uint32_t)j16 % cpp;
    return reinterpret_cast<uint4*>(sCB + pn * PANEL + swz_off((uint32_t)r, c, RBQ));
  };
  mbar_wait(&bars[1], 0, a.status);
  const float cs_i = row_ok ? cs_s[i] : 0.f;
  float tdiag[64];
  float fJ[3] = {0.f, 0.f, 0.f};
  float rpart = 0.f;
  if (row_ok && role == 0) {
    // own sub-block, right to left: E[i,j] = E[i,j+1] a_{j+1}, starting from E[i,i] = 1
    const int ri = i & 63;
    float E = 1.0f;
#pragma unroll
    for (int c = 3; c >= 0; --c) {
      const uint4 w4 = *chunk_ptr(I * 4 + c);
      const uint32_t ww[4] = {w4.x ^ 0x80808080u, w4.y ^ 0x80808080u, w4.z ^ 0x80808080u, w4.w ^ 0x80808080u};
#pragma unroll
      for (int e = 15; e >= 0; --e) {
        const int jj = c * 16 + e;
        float t = 0.f;
        if (jj <= ri) {
          const int j = (I << 6) + jj;
          if (jj < ri) E = __fmul_rn(E, atok_s[j + 1]);
          t = __fmul_rn(unpack_s8(ww[e >> 2], e & 3), __fmul_rn(dt_s[j], E));
        }
        tdiag[jj] = t;
        rpart = fmaxf(rpart, fabsf(t));
      }
    }
  } else if (row_ok) {
#pragma unroll
    for (int J = 0; J < 3; ++J) {
      if (J >= I) break;
      const float f = exp32(__fsub_rn(cs_i, cs_s[J * 64 + 63]));
      fJ[J] = f;
      float bmax = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint4 w4 = *chunk_ptr(J * 4 + c);
        const uint32_t ww[4] = {w4.x ^ 0x80808080u, w4.y ^ 0x80808080u, w4.z ^ 0x80808080u, w4.w ^ 0x80808080u};
        const float* wo = woff_s + J * 64 + c * 16;
#pragma unroll
        for (int e = 0; e < 16; ++e)
          bmax = fmaxf(bmax, fabsf(__fmul_rn(unpack_s8(ww[e >> 2], e & 3), wo[e])));
      }
      rpart = fmaxf(rpart, __fmul_rn(bmax, f));
    }
  }
  part_s[tid] = rpart;
  __syncthreads();
  const float rowmax = fmaxf(part_s[r], part_s[r + 128]);
  const float inv = (rowmax >= 1e-30f) ? __fdiv_rn(127.0f, rowmax) : 0.f;
  if (row_ok && role == 0) {
    if (a.taps.rowmax) a.taps.rowmax[(tok0 + i) * d.H + h] = rowmax;
    int8_t* mq_tap = a.taps.Mq ? a.taps.Mq + ((((i64)b * d.c + k) * d.H + h) * Q + i) * Q + I * 64 : nullptr;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      uint32_t o[4];
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int e = c * 16 + w * 4;
        o[w] = pack4_bits(rne_bits(__fmul_rn(tdiag[e], inv)), rne_bits(__fmul_rn(tdiag[e + 1], inv)),
                          rne_bits(__fmul_rn(tdiag[e + 2], inv)), rne_bits(__fmul_rn(tdiag[e + 3], inv)));
      }
      const uint4 v = make_uint4(o[0], o[1], o[2], o[3]);
      *chunk_ptr(I * 4 + c) = v;
      if (mq_tap) *reinterpret_cast<uint4*>(mq_tap + c * 16) = v;
    }
  } else if (row_ok) {
    int8_t* mq_tap = a.taps.Mq ? a.taps.Mq + ((((i64)b * d.c + k) * d.H + h) * Q + i) * Q : nullptr;
#pragma unroll
    for (int J = 0; J < 3; ++J) {
      if (J >= I) break;
      const float gq = __fmul_rn(fJ[J], inv);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint4* ptr = chunk_ptr(J * 4 + c);
        const uint4 w4 = *ptr;
        const uint32_t ww[4] = {w4.x ^ 0x80808080u, w4.y ^ 0x80808080u, w4.z ^ 0x80808080u, w4.w ^ 0x80808080u};
        const float* wo = woff_s + J * 64 + c * 16;
        uint32_t o[4];
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          uint32_t q4[4];
#pragma unroll
          for (int e = 0; e < 4; ++e)
            q4[e] = rne_bits(__fmul_rn(__fmul_rn(unpack_s8(ww[w], e), wo[w * 4 + e]), gq));
          o[w] = pack4_bits(q4[0], q4[1], q4[2], q4[3]);
        }
        const uint4 v = make_uint4(o[0], o[1], o[2], o[3]);
        *ptr = v;
        if (mq_tap) *reinterpret_cast<uint4*>(mq_tap + J * 64 + c * 16) = v;
      }
    }
    for (int J = I + 1; J < nblk; ++J)  // columns after the row's own sub-block contribute nothing
#pragma unroll
      for (int c = 0; c < 4; ++c) *chunk_ptr(J * 4 + c) = make_uint4(0u, 0u, 0u, 0u);
  }
  fence_async_smem();
  __syncthreads();

  // ---- ChunkScan2 MMA: acc_diag = Mq * xq
  if (tid == 0) {
    mbar_wait(&bars[2], 0, a.status);
    tc_fence_after();
    const uint32_t idesc = idesc_s8(128, 64, 0, 1);
    for (int s = 0; s < KJ / 32; ++s) {
      const uint32_t k0 = 32u * s;
      const uint32_t aaddr = smem_u32(sCB) + (k0 / RBQ) * PANEL + (k0 % RBQ);
      mma_s8_ss(tmem + 64, tile_desc(aaddr, RBQ), tile_desc(smem_u32(sX) + k0 * 64, 64), idesc, s > 0);
    }
    mma_commit(&bars[3]);
  }
  __syncwarp();

  // ---- epilogue: warp w reads TMEM lanes 32 (w % 4) .. +31, columns 32 (w / 4) .. +31
  mbar_wait(&bars[3], 0, a.status);
  mbar_wait(&bars[2], 0, a.status);  // xq rows are read below for the skip term
  tc_fence_after();
  {
    const int q = warp & 3, ch = warp >> 2;
    const int er = q * 32 + lane;        // row of the tile
    const int ei = it * TM + er;         // row of the chunk
    const bool ok = er < TM;
    int acc_o[32], acc_d[32];
    const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(ch * 32);
    tmem_ld32(taddr, acc_o);
    tmem_ld32(taddr + 64, acc_d);
    tmem_ld_wait();
    if (ok) {
      const float dec = exp32(cs_s[ei]);
      const float sm = a.s_cb[g] * fmaxf(part_s[er], part_s[er + 128]) * (1.0f / 127.0f);
      const float Dh = a.D ? a.D[h] : 0.f;
      const uint4 x0 = *reinterpret_cast<const uint4*>(sX + swz_off((uint32_t)ei, (uint32_t)(ch * 2), 64));
      const uint4 x1 = *reinterpret_cast<const uint4*>(sX + swz_off((uint32_t)ei, (uint32_t)(ch * 2 + 1), 64));
      const uint32_t xw[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
      uint8_t* srow = sCB + ch * PANEL + er * 128;
#pragma unroll
      for (int cc = 0; cc < 8; ++cc) {
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int pp = cc * 4 + e, p = ch * 32 + pp;
          const float xv = (float)sx8(xw[pp >> 2], pp & 3);
          v[e] = dec * colA[p] * (float)acc_o[pp] + sm * colB[p] * (float)acc_d[pp] + Dh * colB[p] * xv + colC[p];
        }
        *reinterpret_cast<float4*>(srow + ((cc ^ (er & 7)) << 4)) = make_float4(v[0], v[1], v[2], v[3]);
      }
      if (a.taps.acc_off || a.taps.acc_diag) {
        const i64 o = ((tok0 + ei) * d.H + h) * P + ch * 32;
#pragma unroll
        for (int pp = 0; pp < 32; ++pp) {
          if (a.taps.acc_off) a.taps.acc_off[o + pp] = acc_o[pp];
          if (a.taps.acc_diag) a.taps.acc_diag[o + pp] = acc_d[pp];
        }
      }
    }
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  if (tid == 0) {
    tma_store_3d(&tm_y, sCB, 0, h, (int)(tok0 + it * TM));
    tma_store_3d(&tm_y, sCB + PANEL, 32, h, (int)(tok0 + it * TM));
    tma_store_commit();
    tma_store_wait_read();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

}  // namespace

ssdi8_status_t launch_chunk_scan(const Dims& d, const int8_t* xq, const int8_t* Cq,
                                 const int8_t* CBq, const int8_t* hq, const float* s_x,
                                 const float* s_C, const float* s_cb, const float* s_h,
                                 const float* dt, const float* cs, const float* D,
                                 const float* corr, float* y, int32_t* status, const ScanTaps& taps,
                                 cudaStream_t st) {
  const int TM = d.Q < 128 ? d.Q : 128;
  const uint64_t T = (uint64_t)d.b * d.L;
  CUtensorMap tm_C, tm_h, tm_x, tm_cb, tm_y;
  {
    uint64_t dims[3] = {(uint64_t)d.N, (uint64_t)d.G, T};
    uint64_t str[2] = {(uint64_t)d.N, (uint64_t)d.G * d.N};
    uint32_t box[3] = {(uint32_t)d.N, 1, (uint32_t)TM};
    if (!encode_tensor_map(&tm_C, Cq, 1, 3, dims, str, box, d.N)) return SSDI8_ERR_CUDA;
  }
  {
    uint64_t dims[2] = {(uint64_t)d.N, (uint64_t)d.b * d.c * d.H * d.P};
    uint64_t str[1] = {(uint64_t)d.N};
    uint32_t box[2] = {(uint32_t)d.N, 64};
    if (!encode_tensor_map(&tm_h, hq, 1, 2, dims, str, box, d.N)) return SSDI8_ERR_CUDA;
  }
  {
    uint64_t dims[3] = {(uint64_t)d.P, (uint64_t)d.H, T};
    uint64_t str[2] = {(uint64_t)d.P, (uint64_t)d.H * d.P};
    uint32_t box[3] = {64, 1, (uint32_t)TM};
    if (!encode_tensor_map(&tm_x, xq, 1, 3, dims, str, box, 64)) return SSDI8_ERR_CUDA;
  }
  {
    uint64_t dims[2] = {(uint64_t)d.Q, (uint64_t)d.b * d.c * d.G * d.Q};
    uint64_t str[1] = {(uint64_t)d.Q};
    uint32_t box[2] = {(uint32_t)TM, (uint32_t)TM};
    if (!encode_tensor_map(&tm_cb, CBq, 1, 2, dims, str, box, TM)) return SSDI8_ERR_CUDA;
  }
  {
    uint64_t dims[3] = {(uint64_t)d.P, (uint64_t)d.H, T};
    uint64_t str[2] = {(uint64_t)d.P * 4, (uint64_t)d.H * d.P * 4};
    uint32_t box[3] = {32, 1, (uint32_t)TM};
    if (!encode_tensor_map(&tm_y, y, 4, 3, dims, str, box, 128)) return SSDI8_ERR_CUDA;
  }
  ScanArgs a = {s_x, s_C, s_cb, s_h, dt, cs, D, corr, status, taps, d};
  const size_t smem = SMEM_BYTES + 1024;
  SSDI8_CUDA_CHECK(cudaFuncSetAttribute(chunk_scan_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const unsigned grid = (unsigned)((i64)d.b * d.c * d.H * (d.Q / TM));
  chunk_scan_tc<<<grid, kThreads, smem, st>>>(tm_C, tm_h, tm_x, tm_cb, tm_y, a);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

// ChunkScan1 + ChunkScan2 + output sum (Algorithm 2 modules 5, 6) on tcgen05 tensor cores:
// a persistent, warp-specialised kernel, one CTA per SM, two pipeline stages.
// Per (batch, chunk, head) and 128-row tile of the chunk:
//   acc_off[i,p]  = sum_n Cq[i,n] hq[p,n]                 INT8 MMA, INT32 accumulator in TMEM
//   Mq[i,j]       = per-row re-quantised CBq[i,j] dt_j exp(cs_i - cs_j), j <= i   (see ssdi8.h)
//   acc_diag[i,p] = sum_j Mq[i,j] xq[j,p]                 INT8 MMA, second TMEM accumulator
//   y = exp(cs_i) s_C s_h acc_off + (s_cb rowmax_i / 127) s_x acc_diag + D s_x xq + corr
// Roles: warp 0 issues TMA loads (Cq, hq, CBq K-major; xq MN-major; the per-token scalar pack of
// ChunkCumsum by one bulk copy); warp 1 issues the MMAs; warps 2-5 and 6-9 build Mq in place
// over CBq for even and odd tiles (one thread per output row, no exchange between threads);
// warps 10-13 read the accumulators, form y and store it through swizzled staging with TMA.
// No multicast; every wait is bounded.
#include "kernels.h"
#include "sm100.cuh"

namespace ssdi8 {
namespace {

using namespace sm100;

struct ScanArgs {
  const float* s_x; const float* s_C; const float* s_cb; const float* s_h;
  const float* pack; const float* D; const float* corr;
  int32_t* status;
  ScanTaps taps;
  Dims d;
  int ntiles, per_cta;
};

constexpr int kThreads = 14 * 32;
constexpr uint32_t kTmemCols = 256;  // stage s: acc_off at 128 s, acc_diag at 128 s + 64
// shared memory (bytes, from a 1024-byte aligned base); per stage:
constexpr uint32_t OFF_C = 0;          // [128][N]        Cq tile, K-major
constexpr uint32_t OFF_H = 16384;      // [64][N]         hq tile, K-major
constexpr uint32_t OFF_X = 24576;      // [256][64]       xq rows, MN-major
constexpr uint32_t OFF_CB = 40960;     // 2 x [128][128]  CBq panels -> Mq in place
constexpr uint32_t OFF_TOK = 73728;    // 4 x Q floats: cs, dt, woff, atok (rows 0..3 of the pack)
constexpr uint32_t OFF_PART = 77824;   // [128] rowmax
constexpr uint32_t STAGE = 78848;      // 77 KB
constexpr uint32_t PANEL = 16384;
// after the two stages:
constexpr uint32_t OFF_YST = 2 * STAGE;           // 4 warps x 2 halves x [32][128 B] y staging
constexpr uint32_t OFF_COL = OFF_YST + 32768;     // 4 warps x 4 x [64] per-column factors
constexpr uint32_t OFF_BAR = OFF_COL + 4096;
constexpr uint32_t SMEM_BYTES = OFF_BAR + 256;

enum { B_FULL_CH = 0, B_FULL_CB = 2, B_FULL_X = 4, B_MQ = 6, B_ACC = 8, B_ACC_FREE = 10, B_STAGE_FREE = 12,
       B_COUNT = 14 };

__device__ __forceinline__ float unpack_s8(uint32_t w_xor, int k) {
  // w_xor = word ^ 0x80808080: byte + 128 goes into the mantissa of 1.5 * 2^23
  return __fadd_rn(__uint_as_float(__byte_perm(w_xor, 0x4B400000u, 0x7650u + k)), -12583040.0f);
}
// rne(v) for |v| < 2^22 sits in the low bits of (v + 1.5 * 2^23); callers guarantee |v| < 127.5
__device__ __forceinline__ uint32_t rne_bits(float v) { return __float_as_uint(__fadd_rn(v, 12582912.0f)); }
__device__ __forceinline__ uint32_t pack4_bits(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  return __byte_perm(__byte_perm(a, b, 0x0040u), __byte_perm(c, d, 0x0040u), 0x5410u);
}

struct Tile {
  int b, k, h, g, it, KJ;
  i64 tok0, unit;  // unit = (b*H + h)*c + k
};
__device__ __forceinline__ Tile decode_tile(int t, const Dims& d, int TM, int ntile_per_unit) {
  Tile x;
  x.it = t % ntile_per_unit;
  int u = t / ntile_per_unit;
  x.h = u % d.H; u /= d.H;
  x.k = u % d.c;
  x.b = u / d.c;
  x.g = x.h / (d.H / d.G);
  x.KJ = (x.it + 1) * TM;
  x.tok0 = (i64)x.b * d.L + (i64)x.k * d.Q;
  x.unit = ((i64)x.b * d.H + x.h) * d.c + x.k;
  return x;
}

// ---- one output row of the masked operand, in place over CBq (thread r of the mask group)
__device__ __forceinline__ void mask_row(uint8_t* sCB, const float* tok, float* part_s, int r, int TM,
                                         uint32_t RBQ, const Tile& t, const ScanArgs& a) {
  const int Q = a.d.Q;
  const float* cs_s = tok;
  const float* dt_s = tok + Q;
  const float* woff_s = tok + 2 * Q;
  const float* atok_s = tok + 3 * Q;
  if (r >= TM) return;
  const int i = t.it * TM + r;       // row within the chunk
  const int I = i >> 6;              // its 64-token sub-block
  const int nblk = t.KJ >> 6;        // sub-blocks in the contraction range
  const uint32_t cpp = RBQ >> 4;     // 16-byte chunks per panel row
  auto chunk_ptr = [&](int j16) -> uint4* {
    const uint32_t pn = (uint32_t)j16 / cpp, c = (uint32_t)j16 % cpp;
    return reinterpret_cast<uint4*>(sCB + pn * PANEL + swz_off((uint32_t)r, c, RBQ));
  };
  const float cs_i = cs_s[i];
  float fJ[3] = {0.f, 0.f, 0.f};
  float rowmax = 0.f;
  // earlier sub-blocks: t = cb * woff_j, scaled as a block by f = exp32(cs_i - cs_je)
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
      for (int e = 0; e < 16; ++e) bmax = fmaxf(bmax, fabsf(__fmul_rn(unpack_s8(ww[e >> 2], e & 3), wo[e])));
    }
    rowmax = fmaxf(rowmax, __fmul_rn(bmax, f));
  }
  // own sub-block, right to left: E[i,j] = E[i,j+1] a_{j+1}, starting from E[i,i] = 1
  float tdiag[64];
  {
    const int ri = i & 63;
    float E = 1.0f;
#pragma unroll
    for (int c = 3; c >= 0; --c) {
      const uint4 w4 = *chunk_ptr(I * 4 + c);
      const uint32_t ww[4] = {w4.x ^ 0x80808080u, w4.y ^ 0x80808080u, w4.z ^ 0x80808080u, w4.w ^ 0x80808080u};
#pragma unroll
      for (int e = 15; e >= 0; --e) {
        const int jj = c * 16 + e;
        float tv = 0.f;
        if (jj <= ri) {
          const int j = (I << 6) + jj;
          if (jj < ri) E = __fmul_rn(E, atok_s[j + 1]);
          tv = __fmul_rn(unpack_s8(ww[e >> 2], e & 3), __fmul_rn(dt_s[j], E));
        }
        tdiag[jj] = tv;
        rowmax = fmaxf(rowmax, fabsf(tv));
      }
    }
  }
  part_s[r] = rowmax;
  const float inv = (rowmax >= 1e-30f) ? __fdiv_rn(127.0f, rowmax) : 0.f;
  int8_t* mq_tap = nullptr;
  if (a.taps.Mq) mq_tap = a.taps.Mq + ((((i64)t.b * a.d.c + t.k) * a.d.H + t.h) * Q + i) * Q;
  if (a.taps.rowmax) a.taps.rowmax[(t.tok0 + i) * a.d.H + t.h] = rowmax;
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
    if (mq_tap) *reinterpret_cast<uint4*>(mq_tap + I * 64 + c * 16) = v;
  }
  for (int J = I + 1; J < nblk; ++J)  // columns after the row's own sub-block contribute nothing
#pragma unroll
    for (int c = 0; c < 4; ++c) *chunk_ptr(J * 4 + c) = make_uint4(0u, 0u, 0u, 0u);
}

__global__ void __launch_bounds__(kThreads, 1)
chunk_scan_tc(const __grid_constant__ CUtensorMap tm_C, const __grid_constant__ CUtensorMap tm_h,
              const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_cb,
              const __grid_constant__ CUtensorMap tm_y, const ScanArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const Dims& d = a.d;
  const int Q = d.Q, N = d.N, P = d.P;
  const int TM = Q < 128 ? Q : 128;        // valid rows of a tile
  const int ntpu = Q / TM;                 // tiles per (batch, chunk, head)
  const uint32_t RBN = N, RBQ = TM;        // row bytes of the N-contracted and Q-contracted tiles
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int t_begin = blockIdx.x * a.per_cta;
  const int t_end = min(a.ntiles, t_begin + a.per_cta);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars[B_FULL_CH + s], 1);
      mbar_init(&bars[B_FULL_CB + s], 1);
      mbar_init(&bars[B_FULL_X + s], 1);
      mbar_init(&bars[B_MQ + s], 4);
      mbar_init(&bars[B_ACC + s], 1);
      mbar_init(&bars[B_ACC_FREE + s], 4);
      mbar_init(&bars[B_STAGE_FREE + s], 4);
    }
    fence_mbar_init();
    tma_prefetch_desc(&tm_C); tma_prefetch_desc(&tm_h); tma_prefetch_desc(&tm_x);
    tma_prefetch_desc(&tm_cb); tma_prefetch_desc(&tm_y);
  }
  if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      for (int tix = t_begin, n = 0; tix < t_end; ++tix, ++n) {
        const int s = n & 1, ph = (n >> 1) & 1;
        uint8_t* st = smem + s * STAGE;
        const Tile t = decode_tile(tix, d, TM, ntpu);
        mbar_wait(&bars[B_STAGE_FREE + s], ph ^ 1, a.status);
        mbar_expect_tx(&bars[B_FULL_CH + s], (uint32_t)(TM * N + 64 * N));
        tma_load_3d(st + OFF_C, &tm_C, &bars[B_FULL_CH + s], 0, t.g, (int)(t.tok0 + t.it * TM));
        tma_load_2d(st + OFF_H, &tm_h, &bars[B_FULL_CH + s], 0, (int)((((i64)t.b * d.c + t.k) * d.H + t.h) * P));
        const int npanel = t.KJ / (int)RBQ;
        mbar_expect_tx(&bars[B_FULL_CB + s], (uint32_t)(npanel * TM * RBQ + 4 * Q * 4));
        bulk_load(st + OFF_TOK, a.pack + t.unit * kPackRows * Q, (uint32_t)(4 * Q * 4), &bars[B_FULL_CB + s]);
        for (int pn = 0; pn < npanel; ++pn)
          tma_load_2d(st + OFF_CB + pn * PANEL, &tm_cb, &bars[B_FULL_CB + s], pn * (int)RBQ,
                      (int)((((i64)t.b * d.c + t.k) * d.G + t.g) * Q + t.it * TM));
        mbar_expect_tx(&bars[B_FULL_X + s], (uint32_t)(t.KJ * 64));
        for (int j0 = 0; j0 < t.KJ; j0 += TM)
          tma_load_3d(st + OFF_X + j0 * 64, &tm_x, &bars[B_FULL_X + s], 0, t.h, (int)(t.tok0 + j0));
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_off = idesc_s8(128, 64, 0, 0), idesc_diag = idesc_s8(128, 64, 0, 1);
      for (int tix = t_begin, n = 0; tix < t_end; ++tix, ++n) {
        const int s = n & 1, ph = (n >> 1) & 1;
        const uint32_t sbase = smem_u32(smem + s * STAGE);
        const int KJ = ((tix % ntpu) + 1) * TM;
        const uint32_t acc = tmem + (uint32_t)s * 128u;
        mbar_wait(&bars[B_ACC_FREE + s], ph ^ 1, a.status);
        mbar_wait(&bars[B_FULL_CH + s], ph, a.status);
        tc_fence_after();
        for (int q = 0; q < N / 32; ++q)
          mma_s8_ss(acc, tile_desc(sbase + OFF_C + 32 * q, RBN), tile_desc(sbase + OFF_H + 32 * q, RBN),
                    idesc_off, q > 0);
        mbar_wait(&bars[B_MQ + s], ph, a.status);
        mbar_wait(&bars[B_FULL_X + s], ph, a.status);
        tc_fence_after();
        for (int q = 0; q < KJ / 32; ++q) {
          const uint32_t k0 = 32u * q;
          mma_s8_ss(acc + 64, tile_desc(sbase + OFF_CB + (k0 / RBQ) * PANEL + (k0 % RBQ), RBQ),
                    tile_desc(sbase + OFF_X + k0 * 64, 64), idesc_diag, q > 0);
        }
        mma_commit(&bars[B_ACC + s]);
      }
    }
  } else if (warp < 10) {
    // ------------------------------------------------------------ mask groups (stage = group)
    const int grp = (warp - 2) >> 2;
    const int r = ((warp - 2) & 3) * 32 + lane;
    uint8_t* st = smem + grp * STAGE;
    for (int tix = t_begin + grp, n = grp; tix < t_end; tix += 2, n += 2) {
      const int ph = (n >> 1) & 1;
      const Tile t = decode_tile(tix, d, TM, ntpu);
      mbar_wait(&bars[B_FULL_CB + grp], ph, a.status);
      mask_row(st + OFF_CB, reinterpret_cast<const float*>(st + OFF_TOK),
               reinterpret_cast<float*>(st + OFF_PART), r, TM, RBQ, t, a);
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars[B_MQ + grp]);
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int ew = warp - 10;
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int er = q * 32 + lane;           // row of the tile
    uint8_t* ystage = smem + OFF_YST + ew * 8192;
    float* col = reinterpret_cast<float*>(smem + OFF_COL + ew * 1024);  // A, B, D, C x [64]
    int cur_h = -1;
    for (int tix = t_begin, n = 0; tix < t_end; ++tix, ++n) {
      const int s = n & 1, ph = (n >> 1) & 1;
      const uint8_t* st = smem + s * STAGE;
      const Tile t = decode_tile(tix, d, TM, ntpu);
      if (t.h != cur_h) {
        cur_h = t.h;
        __syncwarp();
        const float sC = a.s_C[t.g], Dh = a.D ? a.D[t.h] : 0.f;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int p = lane + 32 * e, hp = t.h * P + p;
          const float sx = a.s_x[hp];
          col[p] = sC * a.s_h[hp];
          col[64 + p] = sx;
          col[128 + p] = Dh * sx;
          col[192 + p] = a.corr ? a.corr[hp] : 0.f;
        }
        __syncwarp();
      }
      mbar_wait(&bars[B_ACC + s], ph, a.status);
      mbar_wait(&bars[B_MQ + s], ph, a.status);       // rowmax written by the mask group
      mbar_wait(&bars[B_FULL_X + s], ph, a.status);   // xq rows (skip term)
      mbar_wait(&bars[B_FULL_CB + s], ph, a.status);  // cs
      tc_fence_after();
      const bool ok = er < TM;
      const int ei = t.it * TM + er;
      const float* tok = reinterpret_cast<const float*>(st + OFF_TOK);
      const float* part = reinterpret_cast<const float*>(st + OFF_PART);
      const float dec = ok ? exp32(tok[ei]) : 0.f;
      const float sm = ok ? a.s_cb[t.g] * part[er] * (1.0f / 127.0f) : 0.f;
      if (lane == 0 && n > 0) tma_store_wait_read();  // staging of the previous tile has been read
      __syncwarp();
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        int acc_o[32], acc_d[32];
        const uint32_t taddr = tmem + (uint32_t)s * 128u + ((uint32_t)(q * 32) << 16) + (uint32_t)(ch * 32);
        tmem_ld32(taddr, acc_o);
        tmem_ld32(taddr + 64, acc_d);
        tmem_ld_wait();
        if (ok) {
          const uint4 x0 = *reinterpret_cast<const uint4*>(st + OFF_X + swz_off((uint32_t)ei, (uint32_t)(ch * 2), 64));
          const uint4 x1 = *reinterpret_cast<const uint4*>(st + OFF_X + swz_off((uint32_t)ei, (uint32_t)(ch * 2 + 1), 64));
          const uint32_t xw[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
          uint8_t* srow = ystage + ch * 4096 + lane * 128;
#pragma unroll
          for (int cc = 0; cc < 8; ++cc) {
            const int p0 = ch * 32 + cc * 4;
            const float4 cA = *reinterpret_cast<const float4*>(col + p0);
            const float4 cB = *reinterpret_cast<const float4*>(col + 64 + p0);
            const float4 cD = *reinterpret_cast<const float4*>(col + 128 + p0);
            const float4 cC = *reinterpret_cast<const float4*>(col + 192 + p0);
            const float A4[4] = {cA.x, cA.y, cA.z, cA.w}, B4[4] = {cB.x, cB.y, cB.z, cB.w};
            const float D4[4] = {cD.x, cD.y, cD.z, cD.w}, C4[4] = {cC.x, cC.y, cC.z, cC.w};
            float v[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int pp = cc * 4 + e;
              const float xv = (float)sx8(xw[pp >> 2], pp & 3);
              v[e] = fmaf(dec * A4[e], (float)acc_o[pp], fmaf(sm * B4[e], (float)acc_d[pp], fmaf(D4[e], xv, C4[e])));
            }
            *reinterpret_cast<float4*>(srow + ((cc ^ (lane & 7)) << 4)) = make_float4(v[0], v[1], v[2], v[3]);
          }
          if (a.taps.acc_off || a.taps.acc_diag) {
            const i64 o = ((t.tok0 + ei) * d.H + t.h) * P + ch * 32;
#pragma unroll
            for (int pp = 0; pp < 32; ++pp) {
              if (a.taps.acc_off) a.taps.acc_off[o + pp] = acc_o[pp];
              if (a.taps.acc_diag) a.taps.acc_diag[o + pp] = acc_d[pp];
            }
          }
        }
      }
      tc_fence_before();
      fence_async_smem();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&bars[B_ACC_FREE + s]);
        mbar_arrive(&bars[B_STAGE_FREE + s]);
        if (q * 32 < TM) {
          const int row0 = (int)(t.tok0 + t.it * TM + q * 32);
          tma_store_3d(&tm_y, ystage, 0, t.h, row0);
          tma_store_3d(&tm_y, ystage + 4096, 32, t.h, row0);
          tma_store_commit();
        }
      }
    }
    if (lane == 0) tma_store_wait_read();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

}  // namespace

ssdi8_status_t launch_chunk_scan(const Dims& d, const int8_t* xq, const int8_t* Cq,
                                 const int8_t* CBq, const int8_t* hq, const float* s_x,
                                 const float* s_C, const float* s_cb, const float* s_h,
                                 const float* pack, const float* D,
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
    uint32_t box[3] = {32, 1, 32};
    if (!encode_tensor_map(&tm_y, y, 4, 3, dims, str, box, 128)) return SSDI8_ERR_CUDA;
  }
  int dev = 0, sms = 0;
  SSDI8_CUDA_CHECK(cudaGetDevice(&dev));
  SSDI8_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int ntiles = (int)((i64)d.b * d.c * d.H * (d.Q / TM));
  const int ctas = ntiles < sms ? ntiles : sms;
  const int per_cta = (ntiles + ctas - 1) / ctas;
  ScanArgs a = {s_x, s_C, s_cb, s_h, pack, D, corr, status, taps, d, ntiles, per_cta};
  const size_t smem = SMEM_BYTES + 1024;
  SSDI8_CUDA_CHECK(cudaFuncSetAttribute(chunk_scan_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const unsigned grid = (unsigned)((ntiles + per_cta - 1) / per_cta);
  chunk_scan_tc<<<grid, kThreads, smem, st>>>(tm_C, tm_h, tm_x, tm_cb, tm_y, a);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

// ChunkScan1 + ChunkScan2 + output sum with the paper's own ChunkScan2 operand (Section 4.2;
// Algorithm 2, module 6): the masked operand stays in FP16 with the dequantisation scale of CB
// fused into the look-up table,
//   M16[i,j] = half(s_cb CBq[i,j] dt_j exp(cs_i - cs_j)), j <= i,      y_diag = s_x sum_j M16[i,j] xq[j,p],
// instead of the per-row int8 re-quantisation of chunk_scan.cu.  A persistent, warp-specialised
// kernel like that one (28 warps: 2 TMA producers, 2 MMA issuers on alternate tiles, two mask groups
// of 8 warps on alternate tiles, 8 epilogue warps; the FP16 x rows are loaded once per chunk), with
// these differences:
//  * the mask warps write M16 straight into tensor memory (tcgen05.st, thread = row), from where
//    tcgen05.mma.kind::f16 takes it as its A operand: the operand never exists in shared memory,
//    there is no row maximum, no second pass and no zero fill of shared memory;
//  * X enters the MMA as the exact FP16 image of its int8 codes: the codes of a chunk arrive by TMA in
//    the upper half of the chunk's x buffer and the mask group that takes the chunk expands them in
//    place, a row per thread, into the MN-major tile with 128-byte swizzled rows that the MMA reads;
//    the epilogue warps request the codes of the chunk after next when they hand a buffer back;
//    ChunkScan1 stays an int8 MMA;
//  * tensor memory: two accumulator pairs (INT32 C h, FP32 M16 x) and two operand buffers, 512 columns.
// One factor per 16-column sub-block as in chunk_scan.cu: own sub-block by the running product of
// per-token decays, earlier ones woff_j f with f the row's decay to the end of the sub-block before its own
// times ChunkCumsum's tabulated block-to-block decay; a sub-block whose bound
// says every |value| < 2^-25 (half of the smallest FP16 subnormal) is zero, and so is every
// farther one where cs does not increase (p127, see cumsum.cu).  No multicast; bounded waits.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "kernels.h"
#include "scan_common.cuh"
#include "sm100.cuh"

namespace ssdi8 {
namespace {

using namespace sm100;
using namespace scan;

struct ScanArgs {
  const float* s_x; const float* s_C; const float* s_cb; const float* s_h;
  const float* pack; const float* D; const float* corr;
  int32_t* status;
  Dims d;
  UnitWalk w;       // CTA j takes units j, j + grid, j + 2 grid, ...
};

constexpr int kWarps = 28, kThreads = kWarps * 32;
constexpr int kMaskWarp0 = 4, kGroupWarps = 8;
constexpr int kEpiWarp0 = 20, kEpiWarps = 8;
constexpr uint32_t kTmemCols = 512;  // accumulator pair a at 128 a (+0 INT32 C h, +64 FP32 M16 x); operand buffer g at 256 + 128 g
// shared memory (bytes, from a 1024-byte aligned base)
constexpr uint32_t OFF_CB = 0;          // ring of 4: two 2-panel buffers, two 1-panel buffers
constexpr uint32_t OFF_C = 98304;       // [128][N]
constexpr uint32_t OFF_H = 114688;      // [64][N]
constexpr uint32_t OFF_X = 122880;      // ring of 2 x [256][64] fp16 (128-byte rows)
constexpr uint32_t X_BYTES = 32768;
constexpr uint32_t OFF_TOK = OFF_X + 2 * X_BYTES;   // ring of 4 x (5 Q floats: cs, dt, woff, atok, bounds)
constexpr uint32_t TOK_BYTES = 6144;
constexpr uint32_t TOK_SCAL = 5888;   // two scalars of the tile: s_C of the group, D of the head
constexpr uint32_t TOK_COLS = 5120;   // byte offset of the head's s_x, s_h and correction vectors ([64] each) in a slot
constexpr uint32_t OFF_YST = OFF_TOK + 4 * TOK_BYTES;  // 8 warps x [32][64 B] y staging
constexpr uint32_t OFF_BAR = OFF_YST + 16384;
constexpr uint32_t SMEM_BYTES = OFF_BAR + 512;

__device__ __forceinline__ uint32_t cb_offset(int idx) { return scan::cb_offset(OFF_CB, idx); }

// The Cq/hq buffer is single, but its barriers come in pairs indexed by the parity of the tile: the two
// MMA issuers take alternate tiles, and a barrier polled by parity must be seen phase by phase by its
// one waiter (an issuer that skipped a phase would pass its first wait at once).
enum { B_CB_FULL = 0, B_CB_FREE = 4, B_MQ = 8, B_CH_FULL = 12, B_X_FULL = 14, B_X_FREE = 16,
       B_TOK_FULL = 18, B_TOK_FREE = 22, B_ACC = 26, B_ACC_FREE = 28, B_AFREE = 30, B_CH_FREE = 32, B_X_RAW = 34, B_COUNT = 36 };

__device__ __forceinline__ uint32_t half2_bits(float2 v) {
  const __half2 h = __floats2half2_rn(v.x, v.y);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&v)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem], FP16 operands, FP32 accumulator; issued by one thread
__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// instruction descriptor for kind::f16: FP16 A (K-major, in tensor memory) and B, FP32 accumulator
__host__ __device__ constexpr uint32_t idesc_f16(int M, int N, int b_mn_major) {
  return (1u << 4) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ---- the FP16 operand of one tile, written to tensor memory.  A warp owns 32 rows (lane = row =
// TMEM lane, warp index mod 4 = lane quarter) and the 16-column chunks of one parity q2; every
// chunk of that parity in the contraction range gets one collective store of 8 packed words per
// row (zeros where the chunk lies after the row's own, is skipped, or the row is idle).
__device__ __forceinline__ void mask_tile_f16(const uint8_t* sCB, const float* tokbuf, uint32_t a_tmem, int rq,
                                              int q2, int lane, int TM, uint32_t RBQ, const Tile& t,
                                              const ScanArgs& a) {
  const int Q = a.d.Q;
  const float* cs_s = tokbuf;
  const float* dt_s = tokbuf + Q;
  const float* woff_s = tokbuf + 2 * Q;
  const float* atok_s = tokbuf + 3 * Q;
  const float* b127_s = tokbuf + 4 * Q;
  const float* p127_s = b127_s + 16;
  const int r = rq * 32 + lane;
  const bool row_ok = r < TM;
  const int i = t.it * TM + r;       // row within the chunk
  const int I16 = i >> 4, ri = i & 15;
  const int nch = t.KJ >> 4;         // 16-column chunks in the contraction range
  const uint32_t cshift = RBQ == 128 ? 3u : 2u;  // log2(chunks per panel row)
  const uint8_t* const rowbase = sCB + (RBQ == 128 ? (uint32_t)r * 128u : (uint32_t)r * 64u);
  const uint32_t rx = RBQ == 128 ? ((uint32_t)r & 7u) : (((uint32_t)r >> 1) & 3u);  // swizzle term of the row
  auto chunk_ptr = [&](int c) -> const uint4* {
    const uint32_t pn = (uint32_t)c >> cshift, cc = (uint32_t)c & ((1u << cshift) - 1u);
    return reinterpret_cast<const uint4*>(rowbase + pn * PANEL + ((cc ^ rx) << 4));
  };
  const float cs_i = row_ok ? cs_s[i] : 0.f;
  const float scb = a.s_cb[t.h / a.w.hpg];
  // decay to an earlier chunk c: the row's decay to the end of the chunk before its own, times the
  // tabulated decay from there to the end of chunk c (1 for c = I16 - 1)
  const float ri_dec = I16 > 0 ? exp32(__fsub_rn(cs_i, cs_s[I16 * 16 - 1])) : 0.f;
  const float* const gtab = b127_s + 32 + ((I16 * (I16 - 1)) >> 1);
  const float kTiny = 2.9e-8f;       // below 2^-25 = 2.98e-8: rounds to zero in FP16
  const uint32_t lane_addr = a_tmem + ((uint32_t)(rq * 32) << 16);
  bool done = !row_ok;               // this row has nothing (more) to contribute
  // The row's own sub-block, right to left: E[i,i] = 1, E[i,j] = fmul(E[i,j+1], a_{j+1}).  Straight-line
  // code ahead of the walk: a step that a row does not take multiplies by 1 (exact), a column past the
  // diagonal is selected to 0, so the 32 rows of the warp (two sub-blocks, every diagonal position) do
  // not diverge; the walk below only picks the result up when it reaches the sub-block.
  uint32_t own[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
  {
    const uint4 w4 = row_ok ? *chunk_ptr(I16) : make_uint4(0u, 0u, 0u, 0u);
    const uint32_t ww[4] = {w4.x ^ 0x80808080u, w4.y ^ 0x80808080u, w4.z ^ 0x80808080u, w4.w ^ 0x80808080u};
    const int i0 = row_ok ? I16 * 16 : 0;
    const float2 scb2 = make_float2(scb, scb);
    float E = 1.0f;
#pragma unroll
    for (int hf = 1; hf >= 0; --hf) {   // columns 15..8, then 7..0 (the product runs on through both)
      const float4* a4 = reinterpret_cast<const float4*>(atok_s + i0 + 8 * hf);
      const float4* d4 = reinterpret_cast<const float4*>(dt_s + i0 + 8 * hf);
      const float4 A0 = a4[0], A1 = a4[1];
      const float alast = hf ? 1.0f : atok_s[i0 + 8];                      // a_{e+1} for the half's last column
      const float an[8] = {A0.y, A0.z, A0.w, A1.x, A1.y, A1.z, A1.w, alast};
      const float4 D0 = d4[0], D1 = d4[1];
      const float dv[8] = {D0.x, D0.y, D0.z, D0.w, D1.x, D1.y, D1.z, D1.w};
      const int rr = ri - 8 * hf;                                           // columns k <= rr of this half are on or below the diagonal
      float Ev[8];
#pragma unroll
      for (int k = 7; k >= 0; --k) {
        E = __fmul_rn(E, k < rr ? an[k] : 1.0f);
        Ev[k] = E;
      }
#pragma unroll
      for (int k = 0; k < 8; k += 2) {
        const int e = 8 * hf + k;
        const float2 t2 = __fmul2_rn(__fmul2_rn(unpack2(ww[e >> 2], e & 3),
                                                __fmul2_rn(make_float2(dv[k], dv[k + 1]), make_float2(Ev[k], Ev[k + 1]))), scb2);
        own[e >> 1] = half2_bits(make_float2(k <= rr ? t2.x : 0.f, k + 1 <= rr ? t2.y : 0.f));
      }
    }
  }
#pragma unroll 1
  for (int c = ((nch - 1 - q2) & ~1) + q2; c >= 0; c -= 2) {
    uint32_t w8[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
    if (!done && c == I16) {
#pragma unroll
      for (int e = 0; e < 8; ++e) w8[e] = own[e];
    } else if (!done && c < I16) {
      {
        const float g = __fmul_rn(__fmul_rn(ri_dec, gtab[c]), scb);
        if (__fmul_rn(p127_s[c], g) < kTiny) {
          done = true;               // this chunk and every farther one round to zero
        } else if (__fmul_rn(b127_s[c], g) >= kTiny) {
          const float2 g2 = make_float2(g, g);
          const uint4 w4 = *chunk_ptr(c);
          const uint32_t ww[4] = {w4.x ^ 0x80808080u, w4.y ^ 0x80808080u, w4.z ^ 0x80808080u, w4.w ^ 0x80808080u};
          const float4* wo = reinterpret_cast<const float4*>(woff_s + c * 16);
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            const float4 fo = wo[w];
            w8[2 * w] = half2_bits(__fmul2_rn(__fmul2_rn(unpack2(ww[w], 0), make_float2(fo.x, fo.y)), g2));
            w8[2 * w + 1] = half2_bits(__fmul2_rn(__fmul2_rn(unpack2(ww[w], 2), make_float2(fo.z, fo.w)), g2));
          }
        }
      }
    }
    __syncwarp();
    tmem_st8(lane_addr + (uint32_t)(c * 8), w8);
  }
  tmem_st_wait();
}

// The xq rows of a chunk arrive as int8 codes in the upper half of the chunk's x buffer (rows of 64
// bytes from byte 64 Q on) and are expanded in place into the MMA's FP16 operand (rows of 128 bytes,
// 128-byte swizzle, from byte 0) by the mask group that takes the chunk: one row per thread, every
// thread reads its codes, the group meets at its hardware barrier, every thread writes its row.  With
// u = code ^ 0x80 the half with bits 0x6400 | u is 1024 + u exactly, and subtracting 1152 gives the
// code (one byte permute and one packed subtraction per two codes).
__device__ __forceinline__ void x_row_to_half(uint8_t* xb, int r, const uint4 (&w)[4]) {
  const __half2 off = __floats2half2_rn(1152.f, 1152.f);
  uint8_t* row = xb + r * 128;
#pragma unroll
  for (int qd = 0; qd < 4; ++qd) {
    const uint32_t ww[4] = {w[qd].x ^ 0x80808080u, w[qd].y ^ 0x80808080u, w[qd].z ^ 0x80808080u, w[qd].w ^ 0x80808080u};
    uint32_t o[8];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        const uint32_t bits = __byte_perm(ww[k], 0x64646464u, p ? 0x7372u : 0x7170u);  // {0x64, b(2p+1), 0x64, b(2p)}
        const __half2 h = __hsub2(*reinterpret_cast<const __half2*>(&bits), off);
        o[k * 2 + p] = *reinterpret_cast<const uint32_t*>(&h);
      }
    }
    *reinterpret_cast<uint4*>(row + (((2 * qd) ^ (r & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
    *reinterpret_cast<uint4*>(row + (((2 * qd + 1) ^ (r & 7)) << 4)) = make_uint4(o[4], o[5], o[6], o[7]);
  }
}

// CORR: a mean-correction vector is given; YT: format of y (0 binary32, 1 fp16, 2 bf16);
// BIGQ: chunks of 128 tokens or more (128-row tiles, 128-byte CBq rows: the tile geometry is a constant)
template <bool CORR, int YT, bool BIGQ>
__global__ void __launch_bounds__(kThreads, 1)
chunk_scan_f16_tc(const __grid_constant__ CUtensorMap tm_C, const __grid_constant__ CUtensorMap tm_h,
                  const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_cb,
                  const __grid_constant__ CUtensorMap tm_y, const ScanArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const Dims& d = a.d;
  const int Q = d.Q, N = d.N, P = d.P;
  const int TM = BIGQ ? 128 : Q;           // valid rows of a tile
  const int ntpu = BIGQ ? Q / 128 : 1;     // tiles per (batch, chunk, head)
  const uint32_t RBN = N, RBQ = BIGQ ? 128u : (uint32_t)Q;        // row bytes of the N-contracted and Q-contracted int8 tiles
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // tiles of this CTA: its units blockIdx.x, blockIdx.x + gridDim.x, ..., ntpu tiles each
  const int n_end = tiles_of_cta(a.w, (int)blockIdx.x, (int)gridDim.x, ntpu);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);

  if (tid == 0) {
    for (int s = 0; s < 4; ++s) {
      mbar_init(&bars[B_CB_FULL + s], 1);
      mbar_init(&bars[B_CB_FREE + s], kGroupWarps);   // released by the mask group that read it
      mbar_init(&bars[B_MQ + s], kGroupWarps);
      mbar_init(&bars[B_TOK_FULL + s], 1);
      mbar_init(&bars[B_TOK_FREE + s], kEpiWarps);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars[B_CH_FULL + s], 1);
      mbar_init(&bars[B_CH_FREE + s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars[B_X_FULL + s], kGroupWarps);   // the warps of the mask group that expands the rows
      mbar_init(&bars[B_X_RAW + s], 1);
      mbar_init(&bars[B_X_FREE + s], kEpiWarps * ntpu);   // the epilogues of the chunk's tiles
      mbar_init(&bars[B_ACC + s], 1);
      mbar_init(&bars[B_ACC_FREE + s], kEpiWarps);
      mbar_init(&bars[B_AFREE + s], 1);
    }
    fence_mbar_init();
    tma_prefetch_desc(&tm_C); tma_prefetch_desc(&tm_h); tma_prefetch_desc(&tm_x);
    tma_prefetch_desc(&tm_cb); tma_prefetch_desc(&tm_y);
  }
  pdl_launch_dependents();
  if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();   // every role below reads or writes global memory

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer: CBq panels, scalar pack, and the
    // int8 xq rows of each chunk (the mask group that takes the chunk expands them to FP16)
    if (lane == 0) {
      Tile t = decode_unit((int)blockIdx.x, d, TM);
      {   // the int8 xq rows of the first two chunks (both buffers are free); later requests come from the
          // epilogue warps, the moment they have finished with a buffer
        Tile tn = t;
        for (int kc = 0; kc < 2 && kc * ntpu < n_end; ++kc) {
          uint8_t* xb = smem + OFF_X + kc * X_BYTES;
          mbar_expect_tx(&bars[B_X_RAW + kc], (uint32_t)(Q * 64));
          for (int j0 = 0; j0 < Q; j0 += TM)
            tma_load_3d(xb + Q * 64 + j0 * 64, &tm_x, &bars[B_X_RAW + kc], 0, tn.h, (int)(tn.tok0 + j0));
          next_head(tn, d, a.w, TM, ntpu);
        }
      }
#pragma unroll 1
      for (int n = 0; n < n_end; ++n, next_tile(t, d, a.w, TM, ntpu)) {
        const int tg = t.h / a.w.hpg;   // group of the head
        const int ci = cb_index(n, t.it, ntpu), t3 = n & 3;
        const uint32_t ph4 = (n >> 2) & 1;
        mbar_wait_relaxed(&bars[B_CB_FREE + ci], ph4 ^ 1, a.status);
        const int npanel = t.KJ / (int)RBQ;
        mbar_expect_tx(&bars[B_CB_FULL + ci], (uint32_t)(npanel * TM * RBQ));
        for (int pn = 0; pn < npanel; ++pn)
          tma_load_2d(smem + cb_offset(ci) + pn * PANEL, &tm_cb, &bars[B_CB_FULL + ci], pn * (int)RBQ,
                      (int)((((i64)t.b * d.c + t.k) * d.G + tg) * Q + t.it * TM));
        mbar_wait_relaxed(&bars[B_TOK_FREE + t3], ph4 ^ 1, a.status);
        // the scalar pack of the chunk and the head's per-column vectors (the epilogue reads them once per
        // 8-column piece: from global memory each read would be a long-latency load in its chain)
        uint8_t* slot = smem + OFF_TOK + t3 * TOK_BYTES;
        {   // the tile's scalars, fetched here so that their latency is not in the epilogue's chain
          float* sc = reinterpret_cast<float*>(slot + TOK_SCAL);
          sc[0] = a.s_C[tg];
          sc[1] = a.D ? a.D[t.h] : 0.f;
        }
        mbar_expect_tx(&bars[B_TOK_FULL + t3], (uint32_t)(5 * Q * 4 + (CORR ? 3 : 2) * P * 4));
        bulk_load(slot, a.pack + t.unit * kPackRows * Q, (uint32_t)(5 * Q * 4), &bars[B_TOK_FULL + t3]);
        bulk_load(slot + TOK_COLS, a.s_x + t.h * P, (uint32_t)(P * 4), &bars[B_TOK_FULL + t3]);
        bulk_load(slot + TOK_COLS + 256, a.s_h + t.h * P, (uint32_t)(P * 4), &bars[B_TOK_FULL + t3]);
        if (CORR) bulk_load(slot + TOK_COLS + 512, a.corr + t.h * P, (uint32_t)(P * 4), &bars[B_TOK_FULL + t3]);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ TMA producer: Cq, hq
    if (lane == 0) {
      Tile t = decode_unit((int)blockIdx.x, d, TM);
#pragma unroll 1
      for (int n = 0; n < n_end; ++n, next_tile(t, d, a.w, TM, ntpu)) {
        // the MMAs of tile n - 1 (the other issuer's) have read the buffer
        if (n > 0) mbar_wait_relaxed(&bars[B_CH_FREE + ((n - 1) & 1)], ((n - 1) >> 1) & 1, a.status);
        uint64_t* full = &bars[B_CH_FULL + (n & 1)];
        mbar_expect_tx(full, (uint32_t)(TM * N + 64 * N));
        tma_load_3d(smem + OFF_C, &tm_C, full, 0, t.h / a.w.hpg, (int)(t.tok0 + t.it * TM));
        tma_load_2d(smem + OFF_H, &tm_h, full, 0, (int)((((i64)t.b * d.c + t.k) * d.H + t.h) * P));
      }
    }
  } else if (warp == 1 || warp == 3) {
    // ------------------------------------------------------------ MMA issuers: warp 1 takes the even tiles of
    // this CTA, warp 3 the odd ones (a tile is 12 to 20 instructions of 16 tokens each, and issuing one
    // takes a thread about 0.1 us: one issuer alone would set the pace of the kernel)
    if (lane == 0) {
      const int par = warp == 3 ? 1 : 0;
      const uint32_t idesc_off = idesc_s8(128, 64, 0, 0), idesc_diag = idesc_f16(128, 64, 1);
      const uint32_t sbase = smem_u32(smem);
#pragma unroll 1
      for (int n = par; n < n_end; n += 2) {
        const int it = ntpu == 1 ? 0 : (n & 1);   // a CTA's first tile is the first of its unit
        const int ci = cb_index(n, it, ntpu), s2 = n & 1, xs = x_index(n, ntpu);
        const uint32_t ph4 = (n >> 2) & 1, ph2 = (n >> 1) & 1;
        const int KJ = (it + 1) * TM;
        const uint32_t acc = tmem + (uint32_t)s2 * 128u;
        mbar_wait(&bars[B_ACC_FREE + s2], ph2 ^ 1, a.status);
        mbar_wait(&bars[B_CH_FULL + par], ph2, a.status);
        tc_fence_after();
#pragma unroll 1
        for (int q = 0; q < N / 32; ++q)
          mma_s8_ss(acc, tile_desc(sbase + OFF_C + 32 * q, RBN), tile_desc(sbase + OFF_H + 32 * q, RBN),
                    idesc_off, q > 0);
        mma_commit(&bars[B_CH_FREE + par]);
        mbar_wait(&bars[B_MQ + ci], ph4, a.status);        // the operand of this tile is in tensor memory
        mbar_wait(&bars[B_X_FULL + xs], x_phase(n, ntpu), a.status);
        tc_fence_after();
        // 16 tokens per instruction: 8 operand columns and 16 rows of 128 bytes of x
        uint64_t bd = smem_desc(sbase + OFF_X + xs * X_BYTES, 16, 1024, SWZ_128B);
        const uint32_t a_op = tmem + 256u + (uint32_t)s2 * 128u;
#pragma unroll 1
        for (int q = 0; q < KJ / 16; ++q, bd += (16 * 128) >> 4)
          mma_f16_ts(acc + 64, a_op + (uint32_t)(q * 8), bd, idesc_diag, q > 0);
        mma_commit(&bars[B_AFREE + s2]);
        mma_commit(&bars[B_ACC + s2]);
      }
    }
  } else if (warp < kEpiWarp0) {
    // ------------------------------------------------------------ mask warps.  With two tiles per chunk, group g
    // takes the chunks c = g, g + 2, ... of this CTA, both tiles (the second tile of a chunk has three
    // times the sub-blocks of the first: alternating tiles would leave one group with all the large
    // ones); with one tile per chunk the groups alternate tiles.  Tile n uses operand buffer n & 1.
    const int g = (warp - kMaskWarp0) / kGroupWarps;
    const int wg = (warp - kMaskWarp0) % kGroupWarps;
    const int rq = warp & 3;               // TMEM lane quarter of this warp = row quarter of the tile
    const int q2 = wg >> 2;                // chunk parity of this warp
    Tile t = decode_unit((int)blockIdx.x, d, TM);
#pragma unroll 1
    for (int n = 0; n < n_end; ++n, next_tile(t, d, a.w, TM, ntpu)) {
      if ((((ntpu == 1) ? n : (n >> 1)) & 1) != g) continue;
      const int ci = cb_index(n, t.it, ntpu), t3 = n & 3, ob = n & 1;
      const uint32_t ph4 = (n >> 2) & 1;
      // one warp of the group polls, a barrier each on three lanes (the scalar pack, the CBq tile, and
      // the MMAs of tile n - 2, which read the operand buffer); the others wait at a hardware barrier,
      // which costs no issue slots
      if (wg == 0 && lane < 3) {
        const int bi = lane == 0 ? B_TOK_FULL + t3 : lane == 1 ? B_CB_FULL + ci : B_AFREE + ob;
        mbar_wait_relaxed(&bars[bi], lane == 2 ? (((n >> 1) & 1) ^ 1) : ph4, a.status);
      } else if (wg == 0 && lane == 3 && t.it == 0) {
        mbar_wait_relaxed(&bars[B_X_RAW + x_index(n, ntpu)], x_phase(n, ntpu), a.status);   // the chunk's xq codes
      }
      named_bar_sync(1 + g, kGroupWarps * 32);
      if (t.it == 0) {   // first tile of a chunk: the group expands the chunk's xq rows to FP16, a row per thread
        uint8_t* xb = smem + OFF_X + x_index(n, ntpu) * X_BYTES;
        const int r = wg * 32 + lane;
        uint4 w[4];
        if (r < Q) {
#pragma unroll
          for (int qd = 0; qd < 4; ++qd) w[qd] = *reinterpret_cast<const uint4*>(xb + Q * 64 + r * 64 + qd * 16);
        }
        named_bar_sync(1 + g, kGroupWarps * 32);   // every code is in a register: the rows may be overwritten
        if (r < Q) x_row_to_half(xb, r, w);
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars[B_X_FULL + x_index(n, ntpu)]);
      }
      tc_fence_after();
      mask_tile_f16(smem + cb_offset(ci), reinterpret_cast<const float*>(smem + OFF_TOK + t3 * TOK_BYTES),
                    tmem + 256u + (uint32_t)ob * 128u, rq, q2, lane, TM, RBQ, t, a);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&bars[B_MQ + ci]);
        mbar_arrive(&bars[B_CB_FREE + ci]);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps: rows 32 q .., columns 32 ch ..
    const int ew = warp - kEpiWarp0;
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int ch = ew >> 2;                 // column half
    const int er = q * 32 + lane;           // row of the tile
    uint8_t* ystage = smem + OFF_YST + ew * 2048;   // [32][64 B], 64-byte swizzle
    uint8_t* srow = ystage + lane * 64;
    Tile t = decode_unit((int)blockIdx.x, d, TM);
#pragma unroll 1
    for (int n = 0; n < n_end; ++n, next_tile(t, d, a.w, TM, ntpu)) {
      const int s2 = n & 1, t3 = n & 3, xs = x_index(n, ntpu);
      const uint32_t ph4 = (n >> 2) & 1, ph2 = (n >> 1) & 1;
      const float* tok = reinterpret_cast<const float*>(smem + OFF_TOK + t3 * TOK_BYTES);
      const uint8_t* sX = smem + OFF_X + xs * X_BYTES;
      const float4* gsx = reinterpret_cast<const float4*>(smem + OFF_TOK + t3 * TOK_BYTES + TOK_COLS) + ch * 8;
      const float4* gsh = gsx + 16;
      const float4* gco = gsx + 32;
      // three lanes wait side by side: the accumulators, the x rows (skip term), the scalar pack (cs)
      if (ew == 0 && lane < 3) {   // one warp polls, the others wait at a hardware barrier
        const int bi = lane == 0 ? B_ACC + s2 : lane == 1 ? B_X_FULL + xs : B_TOK_FULL + t3;
        mbar_wait_relaxed(&bars[bi], lane == 2 ? ph4 : lane == 1 ? x_phase(n, ntpu) : ph2, a.status);
      }
      named_bar_sync(3, kEpiWarps * 32);
      tc_fence_after();
      const bool ok = er < TM;
      const int ei = t.it * TM + er;
      const float sC = tok[TOK_SCAL / 4], Dh = tok[TOK_SCAL / 4 + 1];
      const float dec = ok ? exp32(tok[ei]) * sC : 0.f;
      const float2 dec2 = make_float2(dec, dec), Dh2 = make_float2(Dh, Dh);
#pragma unroll
      for (int pc = 0; pc < 4; ++pc) {       // 8 columns at a time
        int acc_o[8], acc_d[8];
        const uint32_t taddr = tmem + (uint32_t)s2 * 128u + ((uint32_t)(q * 32) << 16) + (uint32_t)(ch * 32 + pc * 8);
        tmem_ld8(taddr, acc_o);
        tmem_ld8(taddr + 64, acc_d);
        if (YT != 0 ? pc == 0 : (pc & 1) == 0) {
          if (lane == 3) tma_store_wait_read();  // the last store has finished reading the staging tile
          __syncwarp();
        }
        tmem_ld_wait();
        if (ok) {
          // 8 FP16 values of x (exact images of the int8 codes): one 16-byte chunk of the row
          const uint4 xr = *reinterpret_cast<const uint4*>(sX + swz_off((uint32_t)ei, (uint32_t)(ch * 4 + pc), 128));
          const uint32_t xw[4] = {xr.x, xr.y, xr.z, xr.w};
          float2 v[4];
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const float4 sx4 = gsx[pc * 2 + cc], sh4 = gsh[pc * 2 + cc];
            const float4 co4 = CORR ? gco[pc * 2 + cc] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int e2 = 0; e2 < 2; ++e2) {
              const int pp = cc * 4 + e2 * 2;
              const float2 sx2 = e2 ? make_float2(sx4.z, sx4.w) : make_float2(sx4.x, sx4.y);
              const float2 sh2 = e2 ? make_float2(sh4.z, sh4.w) : make_float2(sh4.x, sh4.y);
              const float2 co2 = e2 ? make_float2(co4.z, co4.w) : make_float2(co4.x, co4.y);
              const float2 xv = __half22float2(*reinterpret_cast<const __half2*>(&xw[cc * 2 + e2]));
              const float2 ao = make_float2((float)acc_o[pp], (float)acc_o[pp + 1]);
              const float2 ad = make_float2(__int_as_float(acc_d[pp]), __int_as_float(acc_d[pp + 1]));
              float2 r2 = __ffma2_rn(__fmul2_rn(Dh2, sx2), xv, co2);
              r2 = __ffma2_rn(sx2, ad, r2);
              v[cc * 2 + e2] = __ffma2_rn(__fmul2_rn(dec2, sh2), ao, r2);
            }
            if (YT == 0)
              *reinterpret_cast<float4*>(srow + ((((pc & 1) * 2 + cc) ^ ((lane >> 1) & 3)) << 4)) =
                  make_float4(v[cc * 2].x, v[cc * 2].y, v[cc * 2 + 1].x, v[cc * 2 + 1].y);
          }
          if (YT != 0) {  // 8 values = one 16-byte chunk of the staging row
            uint32_t h[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              if (YT == 1) {
                h[e] = half2_bits(v[e]);
              } else {
                const __nv_bfloat162 bv = __floats2bfloat162_rn(v[e].x, v[e].y);
                h[e] = *reinterpret_cast<const uint32_t*>(&bv);
              }
            }
            *reinterpret_cast<uint4*>(srow + ((pc ^ ((lane >> 1) & 3)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
          }
        }
        if (YT != 0 ? pc == 3 : (pc & 1) == 1) {   // a staging tile is full: 32 columns of 16-bit y, or 16 of binary32
          if (pc == 3) tc_fence_before();
          fence_async_smem();
          __syncwarp();
          if (pc == 3 && lane < 3) {
            mbar_arrive(&bars[lane == 0 ? B_ACC_FREE + s2 : lane == 1 ? B_X_FREE + xs : B_TOK_FREE + t3]);
            // the chunk's last tile: once every epilogue warp is through, its x buffer takes the codes of
            // the chunk after next
            const int n2 = n - (ntpu - 1) + 2 * ntpu;   // first tile of that chunk
            if (ew == 0 && lane == 1 && t.it == ntpu - 1 && n2 < n_end) {
              mbar_wait(&bars[B_X_FREE + xs], x_phase(n, ntpu), a.status);
              Tile tn = t;
              next_unit(tn, d, a.w);
              next_unit(tn, d, a.w);
              uint8_t* xb = smem + OFF_X + xs * X_BYTES;
              mbar_expect_tx(&bars[B_X_RAW + xs], (uint32_t)(Q * 64));
              for (int j0 = 0; j0 < Q; j0 += TM)
                tma_load_3d(xb + Q * 64 + j0 * 64, &tm_x, &bars[B_X_RAW + xs], 0, tn.h, (int)(tn.tok0 + j0));
            }
          } else if (lane == 3 && q * 32 < TM) {
            tma_store_3d(&tm_y, ystage, ch * 32 + (YT != 0 ? 0 : (pc >> 1) * 16), t.h,
                         (int)(t.tok0 + t.it * TM + q * 32));
            tma_store_commit();
          }
        }
      }
    }
    if (lane == 3) tma_store_wait_read();
  }
  tc_fence_before();
  drain_after_timeout(a.status);
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

}  // namespace

ssdi8_status_t launch_chunk_scan_f16(const Dims& d, const int8_t* xq, const int8_t* Cq,
                                     const int8_t* CBq, const int8_t* hq, const float* s_x, const float* s_C,
                                     const float* s_cb, const float* s_h, const float* pack, const float* D,
                                     const float* corr, void* y, int ydt, int32_t* status, cudaStream_t st) {
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
    uint32_t box[3] = {64, 1, (uint32_t)TM};   // int8 codes, plain rows of 64 bytes
    if (!encode_tensor_map(&tm_x, xq, 1, 3, dims, str, box, 0)) return SSDI8_ERR_CUDA;
  }
  {
    uint64_t dims[2] = {(uint64_t)d.Q, (uint64_t)d.b * d.c * d.G * d.Q};
    uint64_t str[1] = {(uint64_t)d.Q};
    uint32_t box[2] = {(uint32_t)TM, (uint32_t)TM};
    if (!encode_tensor_map(&tm_cb, CBq, 1, 2, dims, str, box, TM)) return SSDI8_ERR_CUDA;
  }
  {
    const uint64_t eb = ydt ? 2 : 4;  // bytes per element of y; the staging tile holds 64-byte rows either way
    uint64_t dims[3] = {(uint64_t)d.P, (uint64_t)d.H, T};
    uint64_t str[2] = {(uint64_t)d.P * eb, (uint64_t)d.H * d.P * eb};
    uint32_t box[3] = {ydt ? 32u : 16u, 1, 32};
    if (!encode_tensor_map(&tm_y, y, (int)eb, 3, dims, str, box, 64)) return SSDI8_ERR_CUDA;
  }
  int dev = 0, sms = 0;
  SSDI8_CUDA_CHECK(cudaGetDevice(&dev));
  SSDI8_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  UnitWalk walk;
  int grid_i = 0;
  if (!make_unit_walk(d, TM, sms, &walk, &grid_i)) return SSDI8_ERR_SHAPE;
  ScanArgs a = {s_x, s_C, s_cb, s_h, pack, D, corr, status, d, walk};
  const size_t smem = SMEM_BYTES + 1024;
  const unsigned grid = (unsigned)grid_i;
  auto launch = [&](auto kernel) -> ssdi8_status_t {
    SSDI8_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    return launch_pdl(kernel, dim3(grid), dim3(kThreads), smem, st, tm_C, tm_h, tm_x, tm_cb, tm_y, a) == cudaSuccess ? SSDI8_OK : SSDI8_ERR_CUDA;
  };
  const bool big = d.Q >= 128;
  auto pick = [&](auto corr_c, auto big_c) -> ssdi8_status_t {
    constexpr bool C = decltype(corr_c)::value, B = decltype(big_c)::value;
    if (ydt == 0) return launch(chunk_scan_f16_tc<C, 0, B>);
    if (ydt == 1) return launch(chunk_scan_f16_tc<C, 1, B>);
    return launch(chunk_scan_f16_tc<C, 2, B>);
  };
  ssdi8_status_t ls;
  if (corr)
    ls = big ? pick(std::true_type{}, std::true_type{}) : pick(std::true_type{}, std::false_type{});
  else
    ls = big ? pick(std::false_type{}, std::true_type{}) : pick(std::false_type{}, std::false_type{});
  if (ls != SSDI8_OK) return ls;
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

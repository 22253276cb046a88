// ChunkScan1 + ChunkScan2 + output sum (Algorithm 2 modules 5, 6) on tcgen05 tensor cores:
// a persistent, warp-specialised kernel, one CTA per SM.
// Per (batch, chunk, head) and 128-row tile of the chunk:
//   acc_off[i,p]  = sum_n Cq[i,n] hq[p,n]                 INT8 MMA, INT32 accumulator in TMEM
//   Mq[i,j]       = per-row re-quantised CBq[i,j] dt_j exp(cs_i - cs_j), j <= i   (see ssdi8.h)
//   acc_diag[i,p] = sum_j Mq[i,j] xq[j,p]                 INT8 MMA, second TMEM accumulator
//   y = exp(cs_i) s_C s_h acc_off + (s_cb rowmax_i / 127) s_x acc_diag + D s_x xq + corr
// Roles (28 warps): warps 0, 2, 3 issue the TMA loads (CBq K-major, the per-token scalar pack of
// ChunkCumsum and the head's per-column vectors; Cq, hq K-major; xq MN-major, once per chunk), each
// stream on its own ring; warp 1 issues the MMAs; warps 4-19 build Mq in place over CBq, as two
// groups of 8 warps that take alternate chunks (two threads per output row in adjacent lanes, so a
// warp owns 16 rows and needs no block barrier for the row maximum); warps 20-27 read the
// accumulators, form y and store it through a swizzled staging tile with TMA (128-byte rows), as two
// groups of 4 warps on alternate tiles, so one group's per-tile bookkeeping and waits run under the
// other's arithmetic.  Four accumulator pairs, an xq buffer per chunk (shared by the chunk's two
// tiles) and an 8-deep ring for what the mask warps hand to the epilogue keep the mask and the MMAs
// of the next tiles independent of the epilogue of the current ones.  Every buffer has its own
// "free" barrier, released by whoever reads it last (tcgen05.commit for MMA operands), so loads run
// several tiles ahead.  The kernel is bound by instruction issue, so it is written to issue little:
// in each group one warp polls the mbarriers and the others wait at a hardware barrier, the wait
// loop is one out-of-line function, the tile walk has no divisions, and the code is kept small
// enough for the instruction cache (every role executes different code at the same time).
// No multicast; bounded waits.
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
  uint8_t* y;       // [b*L][H][P] binary32 or 16-bit
  int32_t* status;
  ScanTaps taps;
  Dims d;
  UnitWalk w;       // CTA j takes units j, j + grid, j + 2 grid, ...
};

constexpr int kWarps = 28, kThreads = kWarps * 32;
constexpr int kMaskWarp0 = 4, kGroupWarps = 8;
constexpr int kEpiWarp0 = 20, kEpiWarps = 8, kEpiGroupWarps = 4;
constexpr uint32_t kTmemCols = 512;  // four accumulator pairs: acc_off at 128 a, acc_diag at 128 a + 64
// shared memory (bytes, from a 1024-byte aligned base)
constexpr uint32_t OFF_CB = 0;          // ring of 4: two 2-panel buffers, two 1-panel buffers
constexpr uint32_t OFF_C = 98304;       // [128][N]
constexpr uint32_t OFF_H = 114688;      // [64][N]
constexpr uint32_t OFF_X = 122880;      // ring of 2 x [256][64]: the xq rows of a chunk
constexpr uint32_t OFF_TOK = 155648;    // ring of 4 x (5 Q floats: cs, dt, woff, atok, bounds), read by the mask warps
constexpr uint32_t TOK_BYTES = 5120;
// ring of 8 x what the epilogue needs of a tile: [128] row maxima and [128] cs_i, written by the
// mask warps, and the head's s_x, s_h and correction vectors ([64] each, bulk-loaded).  Eight deep so
// that the mask of a tile never waits for the epilogue of an earlier one.
constexpr uint32_t OFF_ROW = OFF_TOK + 4 * TOK_BYTES;
constexpr uint32_t ROW_BYTES = 2048, ROW_COLS = 1024, ROW_SCAL = 1792;   // scalars: s_C of the group, D of the head, s_cb
constexpr uint32_t OFF_YST = OFF_ROW + 8 * ROW_BYTES;  // 8 warps x [32][128 B] y staging
constexpr uint32_t OFF_BAR = OFF_YST + 32768;
constexpr uint32_t SMEM_BYTES = OFF_BAR + 512;

__device__ __forceinline__ uint32_t cb_offset(int idx) { return scan::cb_offset(OFF_CB, idx); }

enum { B_CB_FULL = 0, B_CB_FREE = 4, B_MQ = 8, B_CH_FULL = 12, B_CH_FREE = 13, B_X_FULL = 14, B_X_FREE = 16,
       B_TOK_FULL = 18, B_TOK_FREE = 22, B_ACC = 26, B_ACC_FREE = 30, B_ROW_FULL = 34, B_ROW_FREE = 42,
       B_COUNT = 50 };


// four codes rn(a g), the exact product rounded once to the nearest integer (ties to even): for
// |a g| < 2^22 that integer sits in the low bits of fma(a, g, 1.5 * 2^23); callers guarantee
// |a g| < 127.5.  (One fused operation by definition: a packed multiply followed by a packed add of
// the rounding constant is not an alternative, the assembler contracts that pair into this very
// fused operation, which differs from the two-step result wherever the rounded product is a tie.)
__device__ __forceinline__ uint32_t pack4_rn_product(float2 a, float2 b, float2 g) {
  const float2 ra = __ffma2_rn(a, g, make_float2(kMagicOut, kMagicOut));
  const float2 rb = __ffma2_rn(b, g, make_float2(kMagicOut, kMagicOut));
  return __byte_perm(__byte_perm(__float_as_uint(ra.x), __float_as_uint(ra.y), 0x0040u),
                     __byte_perm(__float_as_uint(rb.x), __float_as_uint(rb.y), 0x0040u), 0x5410u);
}

// ---- the masked operand of one tile, in place over CBq.  Two threads per output row, in
// adjacent lanes, so a warp owns 16 rows that share their own sub-block I16 = i / 16 (the walk
// below is warp-uniform up to the skip tests) and the row maximum needs one shuffle, no block
// barrier.  Chunk I16 (16 columns) is the row's own sub-block: running product of per-token
// decays, columns split 8/8 between the two threads (the one with the lower columns first runs
// the product through the upper ones).  Earlier chunks use the column weights woff and one
// factor f = exp32(cs_i - cs_ce) per chunk and are dealt alternately; later chunks are zero.
//
// Work that decides no output bit is skipped, nearest chunk first.  b127[c] bounds |cb woff| of
// chunk c, so a chunk with fmul(b127[c], f) <= (running maximum) cannot raise the row maximum,
// and one with fmul(b127[c], f inv) < 1/2 rounds to zero everywhere.  p127[c] bounds b127 of
// chunks 0..c with a 1e-5 slack; where cs does not increase along the chunk, f of a farther
// chunk is at most f of a nearer one (up to the few 1e-7 of exp32's error, inside the slack),
// so the same two tests on p127[c] end the walk for all farther chunks at once.  (p127 is +inf
// where cs is not monotone: the walk then visits every chunk.)
template <bool TAPS>
__device__ __forceinline__ void mask_tile(uint8_t* sCB, const float* tokbuf, float* rowbuf, int rb, int lane, int TM, uint32_t RBQ,
                                          const Tile& t, const ScanArgs& a) {
  const int Q = a.d.Q;
  const float* cs_s = tokbuf;
  const float* dt_s = tokbuf + Q;
  const float* woff_s = tokbuf + 2 * Q;
  const float* atok_s = tokbuf + 3 * Q;
  const float* b127_s = tokbuf + 4 * Q;
  const float* p127_s = b127_s + 16;
  const int r = rb * 16 + (lane >> 1), q2 = lane & 1;   // the warp's block of 16 rows
  if (r >= TM) return;               // whole warps (TM is a multiple of 16)
  const int i = t.it * TM + r;       // row within the chunk
  const int I16 = i >> 4, ri = i & 15;
  const uint32_t cshift = RBQ == 128 ? 3u : 2u;  // log2(chunks per panel row)
  uint8_t* const rowbase = sCB + (RBQ == 128 ? (uint32_t)r * 128u : (uint32_t)r * 64u);
  const uint32_t rx = RBQ == 128 ? ((uint32_t)r & 7u) : (((uint32_t)r >> 1) & 3u);  // swizzle term of the row
  auto chunk_ptr = [&](int c) -> uint4* {
    const uint32_t pn = (uint32_t)c >> cshift, cc = (uint32_t)c & ((1u << cshift) - 1u);
    return reinterpret_cast<uint4*>(rowbase + pn * PANEL + ((cc ^ rx) << 4));
  };
  const float cs_i = cs_s[i];
  const int c_first = I16 - 1 - q2;  // nearest earlier chunk of this thread (may be < 0)
  float tv[8];                       // t of this thread's half of the row's own sub-block
  float rpart = 0.f;
  // f of an earlier chunk c: the row's decay to the end of the chunk before its own, times the tabulated
  // decay from there to the end of chunk c (gtab[c]; 1 for c = I16 - 1)
  const float ri_dec = I16 > 0 ? exp32(__fsub_rn(cs_i, cs_s[I16 * 16 - 1])) : 0.f;
  const float* const gtab = b127_s + 32 + ((I16 * (I16 - 1)) >> 1);
  uint2* const own_ptr = reinterpret_cast<uint2*>(chunk_ptr(I16)) + q2;
  {
    // own sub-block, right to left: E[i,i] = 1, E[i,j] = fmul(E[i,j+1], a_{j+1}).  Straight-line code:
    // a step that a row does not take multiplies by 1 (exact), a column past the diagonal is
    // selected to 0, so the 16 rows of the warp, which all stop at different columns, do not diverge.
    const uint2 w2 = *own_ptr;
    const uint32_t ww[2] = {w2.x ^ 0x80808080u, w2.y ^ 0x80808080u};
    const float* ab = atok_s + I16 * 16;   // a_m of the sub-block at ab[m]
    const int e0 = q2 * 8;
    float E = 1.0f;
    {
      // the thread with the lower columns first runs the product through the upper ones: a_15 .. a_9
      const float4 p2 = *reinterpret_cast<const float4*>(ab + 8), p3 = *reinterpret_cast<const float4*>(ab + 12);
      const float au[7] = {p2.y, p2.z, p2.w, p3.x, p3.y, p3.z, p3.w};   // a_9 .. a_15
      const int lim = q2 ? 0 : ri;         // steps m <= lim are taken
#pragma unroll
      for (int m = 15; m >= 9; --m) E = __fmul_rn(E, m <= lim ? au[m - 9] : 1.0f);
    }
    const float4 h0 = *reinterpret_cast<const float4*>(ab + e0), h1 = *reinterpret_cast<const float4*>(ab + e0 + 4);
    const float hn[8] = {h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w, ab[e0 + 8]};   // a_{e0+k+1}; the last one is never taken when e0 = 8
    const float4 d0 = *reinterpret_cast<const float4*>(dt_s + I16 * 16 + e0);
    const float4 d1 = *reinterpret_cast<const float4*>(dt_s + I16 * 16 + e0 + 4);
    const float dv[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
    const int rr = ri - e0;                // this thread's columns k <= rr are on or below the diagonal
    float Ev[8];
#pragma unroll
    for (int k = 7; k >= 0; --k) {
      E = __fmul_rn(E, k < rr ? hn[k] : 1.0f);
      Ev[k] = E;
    }
#pragma unroll
    for (int k = 0; k < 8; k += 2) {
      const float2 t2 = __fmul2_rn(unpack2(ww[k >> 2], k & 3),
                                   __fmul2_rn(make_float2(dv[k], dv[k + 1]), make_float2(Ev[k], Ev[k + 1])));
      tv[k] = k <= rr ? t2.x : 0.f;
      tv[k + 1] = k + 1 <= rr ? t2.y : 0.f;
      rpart = fmaxf(fmaxf(rpart, fabsf(tv[k])), fabsf(tv[k + 1]));
    }
  }
  // Both walks below are warp-uniform: every lane steps through the same iterations (chunk
  // c_first - 2 it; the thread of a pair that starts one chunk farther runs out one step earlier) and
  // the skip tests are taken by vote, so the 16 rows of the warp do not diverge; a lane whose own test
  // says "skip" computes along with the others, which changes nothing (its values cannot raise the
  // row maximum, or round to zero).
  constexpr uint32_t kAll = 0xffffffffu;
  const int nit = (I16 + 1) >> 1;
  bool live = true;                  // this row has not reached its prefix bound yet
#pragma unroll 1
  for (int itc = 0; itc < nit; ++itc) {
    const int c = c_first - 2 * itc;
    live = live && c >= 0;
    if (!__any_sync(kAll, live)) break;
    const int cc = c < 0 ? 0 : c;
    const float f = __fmul_rn(ri_dec, gtab[cc]);
    if (rpart >= 1e-30f && __fmul_rn(p127_s[cc], f) <= rpart) live = false;  // nor can any farther chunk
    const bool need = live && !(__fmul_rn(b127_s[cc], f) <= rpart);
    if (!__any_sync(kAll, need)) continue;
    const uint4 w4 = *chunk_ptr(cc);
    const uint32_t ww[4] = {w4.x ^ 0x80808080u, w4.y ^ 0x80808080u, w4.z ^ 0x80808080u, w4.w ^ 0x80808080u};
    const float4* wo = reinterpret_cast<const float4*>(woff_s + cc * 16);
    float bmax = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float4 o = wo[w];
      const float2 t0 = __fmul2_rn(unpack2(ww[w], 0), make_float2(o.x, o.y));
      const float2 t1 = __fmul2_rn(unpack2(ww[w], 2), make_float2(o.z, o.w));
      bmax = fmaxf(fmaxf(bmax, fabsf(t0.x)), fabsf(t0.y));
      bmax = fmaxf(fmaxf(bmax, fabsf(t1.x)), fabsf(t1.y));
    }
    if (need) rpart = fmaxf(rpart, __fmul_rn(bmax, f));
  }
  const float rowmax = fmaxf(rpart, __shfl_xor_sync(0xffffffffu, rpart, 1));
  const float inv = (rowmax >= 1e-30f) ? __fdiv_rn(127.0f, rowmax) : 0.f;
  int8_t* mq_tap = nullptr;
  if (TAPS && a.taps.Mq) mq_tap = a.taps.Mq + ((((i64)t.b * a.d.c + t.k) * a.d.H + t.h) * Q + i) * Q;
  if (q2 == 0) {
    rowbuf[r] = rowmax;                 // read by the epilogue warps, with cs_i (they take its
    rowbuf[128 + r] = cs_i;             // exponential: the mask warps set the pace of the kernel)
    if (TAPS && a.taps.rowmax) a.taps.rowmax[(t.tok0 + i) * a.d.H + t.h] = rowmax;
  }
  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
  // (the chunks after the row's own arrive as zeros: ChunkBMM writes them so)
  {
    const float2 inv2 = make_float2(inv, inv);
    uint2 v;
    v.x = pack4_rn_product(make_float2(tv[0], tv[1]), make_float2(tv[2], tv[3]), inv2);
    v.y = pack4_rn_product(make_float2(tv[4], tv[5]), make_float2(tv[6], tv[7]), inv2);
    *own_ptr = v;
    if (TAPS && mq_tap) *reinterpret_cast<uint2*>(mq_tap + I16 * 16 + q2 * 8) = v;
  }
  bool dead = false;                 // this chunk and every farther one round to zero in this row
  int itc = 0;
#pragma unroll 1
  for (; itc < nit; ++itc) {
    const int c = c_first - 2 * itc;
    const bool valid = c >= 0;
    const int cc = valid ? c : 0;
    // once no row of the warp has a chunk left that does not round to zero, what remains is zero fill
    if (!__any_sync(kAll, valid && !dead)) break;
    uint4* ptr = chunk_ptr(cc);
    uint4 v = zero4;
    {
      const float f = __fmul_rn(ri_dec, gtab[cc]);
      const float g = __fmul_rn(f, inv);
      if (__fmul_rn(p127_s[cc], g) < 0.5f) dead = true;
      const bool need = valid && !dead && __fmul_rn(b127_s[cc], g) >= 0.5f;
      if (__any_sync(kAll, need)) {
        const float2 g2 = make_float2(g, g);
        const uint4 w4 = *ptr;
        const uint32_t ww[4] = {w4.x ^ 0x80808080u, w4.y ^ 0x80808080u, w4.z ^ 0x80808080u, w4.w ^ 0x80808080u};
        const float4* wo = reinterpret_cast<const float4*>(woff_s + cc * 16);
        uint32_t o[4];
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const float4 fo = wo[w];
          o[w] = pack4_rn_product(__fmul2_rn(unpack2(ww[w], 0), make_float2(fo.x, fo.y)),
                                  __fmul2_rn(unpack2(ww[w], 2), make_float2(fo.z, fo.w)), g2);
        }
        if (need) v = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
    if (valid) {
      *ptr = v;
      if (TAPS && mq_tap) *reinterpret_cast<uint4*>(mq_tap + c * 16) = v;
    }
  }
  // the chunks farther left are zeros in every row of the warp
#pragma unroll 1
  for (int c = c_first - 2 * itc; c >= 0; c -= 2) {
    *chunk_ptr(c) = zero4;
    if (TAPS && mq_tap) *reinterpret_cast<uint4*>(mq_tap + c * 16) = zero4;
  }
}

// CORR: a mean-correction vector is given; TAPS: intermediate tensors are written out (tests);
// YT: format of y (0 binary32, 1 fp16, 2 bf16: rounded to nearest even on the way to the staging tile);
// BIGQ: chunks of 128 tokens or more (128-row tiles with 128-byte CBq rows: the tile geometry, which
// every role's address arithmetic depends on, is then known at compile time)
template <bool CORR, bool TAPS, int YT, bool BIGQ>
__global__ void __launch_bounds__(kThreads, 1)
chunk_scan_tc(const __grid_constant__ CUtensorMap tm_C, const __grid_constant__ CUtensorMap tm_h,
              const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_cb,
              const __grid_constant__ CUtensorMap tm_y, const ScanArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const Dims& d = a.d;
  const int Q = d.Q, N = d.N, P = d.P;
  const int TM = BIGQ ? 128 : Q;           // valid rows of a tile
  const int ntpu = BIGQ ? Q / 128 : 1;     // tiles per (batch, chunk, head)
  const uint32_t RBN = N, RBQ = BIGQ ? 128u : (uint32_t)Q;   // row bytes of the N-contracted and Q-contracted tiles
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // tiles of this CTA: its units blockIdx.x, blockIdx.x + gridDim.x, ..., ntpu tiles each
  const int n_end = tiles_of_cta(a.w, (int)blockIdx.x, (int)gridDim.x, ntpu);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  Tile* first_tile = reinterpret_cast<Tile*>(bars + B_COUNT + 2);   // 416 .. 464 of the 512 bytes

  if (tid == 0) {
    for (int s = 0; s < 4; ++s) {
      mbar_init(&bars[B_CB_FULL + s], 1);
      mbar_init(&bars[B_CB_FREE + s], 1);
      mbar_init(&bars[B_MQ + s], kGroupWarps);
      mbar_init(&bars[B_TOK_FULL + s], 1);
      mbar_init(&bars[B_TOK_FREE + s], kGroupWarps);
      mbar_init(&bars[B_ACC + s], 1);
      mbar_init(&bars[B_ACC_FREE + s], kEpiGroupWarps);
    }
    for (int s = 0; s < 8; ++s) {
      mbar_init(&bars[B_ROW_FULL + s], 1 + kGroupWarps);   // the column vectors and the mask warps' row scalars
      mbar_init(&bars[B_ROW_FREE + s], kEpiGroupWarps);
    }
    mbar_init(&bars[B_CH_FULL], 1);
    mbar_init(&bars[B_CH_FREE], 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars[B_X_FULL + s], 1);
      mbar_init(&bars[B_X_FREE + s], ntpu == 1 ? kEpiGroupWarps : kEpiWarps);  // the epilogues of the chunk's tiles
    }
    fence_mbar_init();
    tma_prefetch_desc(&tm_C); tma_prefetch_desc(&tm_h); tma_prefetch_desc(&tm_x);
    tma_prefetch_desc(&tm_cb); tma_prefetch_desc(&tm_y);
    *first_tile = decode_unit((int)blockIdx.x, d, TM);
  }
  pdl_launch_dependents();
  if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();   // every role below reads or writes global memory

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer: CBq panels + scalar pack
    if (lane == 0) {
      Tile t = *first_tile;
#pragma unroll 1
      for (int n = 0; n < n_end; ++n, next_tile(t, d, a.w, TM, ntpu)) {
        const int tg = t.h / a.w.hpg;   // group of the head (one division per tile in this one thread)
        const int ci = cb_index(n, t.it, ntpu), t3 = n & 3;
        const uint32_t ph4 = (n >> 2) & 1, ph3 = (n >> 2) & 1;
        mbar_wait_relaxed(&bars[B_CB_FREE + ci], ph4 ^ 1, a.status);
        const int npanel = t.KJ / (int)RBQ;
        mbar_expect_tx(&bars[B_CB_FULL + ci], (uint32_t)(npanel * TM * RBQ));
        for (int pn = 0; pn < npanel; ++pn)
          tma_load_2d(smem + cb_offset(ci) + pn * PANEL, &tm_cb, &bars[B_CB_FULL + ci], pn * (int)RBQ,
                      (int)((((i64)t.b * d.c + t.k) * d.G + tg) * Q + t.it * TM));
        mbar_wait_relaxed(&bars[B_TOK_FREE + t3], ph3 ^ 1, a.status);
        // the scalar pack of the chunk for the mask warps
        mbar_expect_tx(&bars[B_TOK_FULL + t3], (uint32_t)(5 * Q * 4));
        bulk_load(smem + OFF_TOK + t3 * TOK_BYTES, a.pack + t.unit * kPackRows * Q, (uint32_t)(5 * Q * 4),
                  &bars[B_TOK_FULL + t3]);
        // the head's per-column vectors for the epilogue (read once per 8-column piece: from global
        // memory each read would be a long-latency load in its chain)
        const int r8 = n & 7;
        mbar_wait_relaxed(&bars[B_ROW_FREE + r8], ((n >> 3) & 1) ^ 1, a.status);
        uint8_t* cols = smem + OFF_ROW + r8 * ROW_BYTES + ROW_COLS;
        {   // the tile's three scalars, fetched here so that their latency is not in the epilogue's chain
          float* sc = reinterpret_cast<float*>(smem + OFF_ROW + r8 * ROW_BYTES + ROW_SCAL);
          sc[0] = a.s_C[tg];
          sc[1] = a.D ? a.D[t.h] : 0.f;
          sc[2] = a.s_cb[tg];
        }
        mbar_expect_tx(&bars[B_ROW_FULL + r8], (uint32_t)((CORR ? 3 : 2) * P * 4));   // (an arrival: releases the stores above)
        bulk_load(cols, a.s_x + t.h * P, (uint32_t)(P * 4), &bars[B_ROW_FULL + r8]);
        bulk_load(cols + 256, a.s_h + t.h * P, (uint32_t)(P * 4), &bars[B_ROW_FULL + r8]);
        if (CORR) bulk_load(cols + 512, a.corr + t.h * P, (uint32_t)(P * 4), &bars[B_ROW_FULL + r8]);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ TMA producer: Cq, hq
    if (lane == 0) {
      Tile t = *first_tile;
#pragma unroll 1
      for (int n = 0; n < n_end; ++n, next_tile(t, d, a.w, TM, ntpu)) {
        mbar_wait_relaxed(&bars[B_CH_FREE], (n & 1) ^ 1, a.status);
        mbar_expect_tx(&bars[B_CH_FULL], (uint32_t)(TM * N + 64 * N));
        tma_load_3d(smem + OFF_C, &tm_C, &bars[B_CH_FULL], 0, t.h / a.w.hpg, (int)(t.tok0 + t.it * TM));
        tma_load_2d(smem + OFF_H, &tm_h, &bars[B_CH_FULL], 0, (int)((((i64)t.b * d.c + t.k) * d.H + t.h) * P));
      }
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------ TMA producer: xq rows
    if (lane == 0) {
      Tile t = *first_tile;
#pragma unroll 1
      for (int n = 0; n < n_end; ++n, next_tile(t, d, a.w, TM, ntpu)) {
        if (t.it != 0) continue;   // the chunk's rows were loaded with its first tile
        const int xs = x_index(n, ntpu);
        mbar_wait_relaxed(&bars[B_X_FREE + xs], x_phase(n, ntpu) ^ 1, a.status);
        mbar_expect_tx(&bars[B_X_FULL + xs], (uint32_t)(Q * 64));
        for (int j0 = 0; j0 < Q; j0 += TM)
          tma_load_3d(smem + OFF_X + xs * 16384 + j0 * 64, &tm_x, &bars[B_X_FULL + xs], 0, t.h, (int)(t.tok0 + j0));
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_off = idesc_s8(128, 64, 0, 0), idesc_diag = idesc_s8(128, 64, 0, 1);
      const uint32_t sbase = smem_u32(smem);
#pragma unroll 1
      for (int n = 0; n < n_end; ++n) {
        const int it = ntpu == 1 ? 0 : (n & 1);   // a CTA's first tile is the first of its unit
        const int ci = cb_index(n, it, ntpu), a4 = n & 3, xs = x_index(n, ntpu);
        const uint32_t ph4 = (n >> 2) & 1;
        const int KJ = (it + 1) * TM;
        const uint32_t acc = tmem + (uint32_t)a4 * 128u;
        mbar_wait(&bars[B_ACC_FREE + a4], ph4 ^ 1, a.status);
        mbar_wait(&bars[B_CH_FULL], n & 1, a.status);
        tc_fence_after();
        // descriptors advance by a constant per 32-byte K step (their low bits are the address >> 4):
        // this thread's issue time is on the path from a freed accumulator to the next epilogue
        {
          uint64_t da = tile_desc(sbase + OFF_C, RBN), db = tile_desc(sbase + OFF_H, RBN);
#pragma unroll 1
          for (int q = 0; q < N / 32; ++q, da += 2, db += 2) mma_s8_ss(acc, da, db, idesc_off, q > 0);
        }
        mma_commit(&bars[B_CH_FREE]);
        mbar_wait(&bars[B_MQ + ci], ph4, a.status);
        mbar_wait(&bars[B_X_FULL + xs], x_phase(n, ntpu), a.status);
        tc_fence_after();
        {
          uint64_t db = tile_desc(sbase + OFF_X + xs * 16384, 64);
          uint32_t first = 0;
#pragma unroll 1
          for (uint32_t pn = 0; pn < (uint32_t)KJ / RBQ; ++pn) {     // panels of RBQ columns of Mq
            uint64_t da = tile_desc(sbase + cb_offset(ci) + pn * PANEL, RBQ);
#pragma unroll 1
            for (uint32_t q = 0; q < RBQ / 32; ++q, da += 2, db += (32 * 64) >> 4) {
              mma_s8_ss(acc + 64, da, db, idesc_diag, first);
              first = 1;
            }
          }
        }
        mma_commit(&bars[B_CB_FREE + ci]);
        mma_commit(&bars[B_ACC + a4]);
      }
    }
  } else if (warp < kEpiWarp0) {
    // ------------------------------------------------------------ mask warps.  With two tiles per chunk, group g
    // takes the chunks c = g, g + 2, ... of this CTA, both tiles: warp w builds the 16-row block w of the
    // first tile and block 7 - w of the second, which is the same number of 16-column sub-blocks for every
    // warp (the causal rows grow with the row index).  With one tile per chunk the groups alternate tiles.
    const int g = (warp - kMaskWarp0) / kGroupWarps;
    const int w = (warp - kMaskWarp0) % kGroupWarps;
    Tile t = *first_tile;
    if (g) next_head(t, d, a.w, TM, ntpu);
#pragma unroll 1
    for (int n = g * ntpu; n < n_end; ++n) {
      const int ci = cb_index(n, t.it, ntpu), t3 = n & 3, r8 = n & 7;
      const uint32_t ph4 = (n >> 2) & 1;
      const int rb = t.it ? kGroupWarps - 1 - w : w;
      // one warp of the group polls (the scalar pack, the CBq tile, and the epilogue of the tile that
      // used the row slot); the others wait at a hardware barrier, which costs no issue slots
      if (w == 0 && lane < 3) {
        const int bi = lane == 0 ? B_TOK_FULL + t3 : lane == 1 ? B_CB_FULL + ci : B_ROW_FREE + r8;
        mbar_wait_relaxed(&bars[bi], lane == 2 ? (((n >> 3) & 1) ^ 1) : ph4, a.status);
      }
      named_bar_sync(1 + g, kGroupWarps * 32);
      mask_tile<TAPS>(smem + cb_offset(ci), reinterpret_cast<const float*>(smem + OFF_TOK + t3 * TOK_BYTES),
                      reinterpret_cast<float*>(smem + OFF_ROW + r8 * ROW_BYTES), rb, lane, TM, RBQ, t, a);
      fence_async_smem();
      __syncwarp();
      if (lane < 3) mbar_arrive(&bars[lane == 0 ? B_MQ + ci : lane == 1 ? B_TOK_FREE + t3 : B_ROW_FULL + r8]);
      if (t.it + 1 < ntpu) {   // the chunk's second tile
        t.it = 1;
        t.KJ = 2 * TM;
      } else {                 // skip the other group's chunk (or tile)
        next_head(t, d, a.w, TM, ntpu);
        next_head(t, d, a.w, TM, ntpu);
        n += ntpu;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps: two groups of four take
    // alternate tiles; warp q of a group owns rows 32 q .. of the tile and all 64 columns
    const int ew = warp - kEpiWarp0;
    const int eg = ew / kEpiGroupWarps;     // group: tiles n = eg, eg + 2, ...
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int er = q * 32 + lane;           // row of the tile
    uint8_t* ystage = smem + OFF_YST + ew * 4096;   // [32][128 B], 16-byte chunks swizzled by the row
    uint8_t* srow = ystage + lane * 128;
    constexpr int PPR = YT ? 8 : 4;         // 8-column pieces per round (128 bytes of y per row)
    Tile t = *first_tile;
    if (eg) next_tile(t, d, a.w, TM, ntpu);
#pragma unroll 1
    for (int n = eg; n < n_end; n += 2) {
      const int ci = cb_index(n, t.it, ntpu), a4 = n & 3, xs = x_index(n, ntpu);
      const uint32_t ph4 = (n >> 2) & 1;
      const float* row = reinterpret_cast<const float*>(smem + OFF_ROW + (n & 7) * ROW_BYTES);
      const uint8_t* sX = smem + OFF_X + xs * 16384;
      const float4* ssx = reinterpret_cast<const float4*>(row + ROW_COLS / 4);
      const float4* ssh = ssx + 16;
      const float4* sco = ssx + 32;
      // three lanes of one warp of the group poll side by side, one barrier each: the accumulators, the
      // xq rows (skip term), and the row slot (the head's column vectors and the row scalars written by
      // the mask warps; not the mask barrier of the CBq buffer, which may complete a second time before
      // this group gets here); the other warps wait at a hardware barrier, which costs no issue slots
      if (q == 0 && lane < 3) {
        const int bi = lane == 0 ? B_ACC + a4 : lane == 1 ? B_X_FULL + xs : B_ROW_FULL + (n & 7);
        const uint32_t bp = lane == 0 ? ph4 : lane == 1 ? x_phase(n, ntpu) : ((n >> 3) & 1);
        mbar_wait_relaxed(&bars[bi], bp, a.status);
      }
      named_bar_sync(3 + eg, kEpiGroupWarps * 32);
      tc_fence_after();
      const bool ok = er < TM;
      const int ei = t.it * TM + er;
      const float sC = row[ROW_SCAL / 4], Dh = row[ROW_SCAL / 4 + 1], scb = row[ROW_SCAL / 4 + 2];
      const float dec = ok ? exp32(row[128 + er]) * sC : 0.f;
      const float sm = ok ? scb * row[er] * (1.0f / 127.0f) : 0.f;
      const float2 dec2 = make_float2(dec, dec), sm2 = make_float2(sm, sm), Dh2 = make_float2(Dh, Dh);
      const uint32_t tbase = tmem + (uint32_t)a4 * 128u + ((uint32_t)(q * 32) << 16);
#pragma unroll 4                           // (a round of 32 columns per iteration: the piece index folds into addresses)
      for (int pc = 0; pc < 8; ++pc) {       // 8 columns at a time (keeps the accumulators in registers)
        int acc_o[8], acc_d[8];
        tmem_ld8(tbase + pc * 8, acc_o);
        tmem_ld8(tbase + 64 + pc * 8, acc_d);
        if ((pc & (PPR - 1)) == 0) {         // the last store has finished reading the staging tile
          if (lane == 3) tma_store_wait_read();
          __syncwarp();
        }
        tmem_ld_wait();
        if (ok) {
          const uint2 xr = *reinterpret_cast<const uint2*>(sX + swz_off((uint32_t)ei, (uint32_t)(pc >> 1), 64) + (pc & 1) * 8);
          const uint32_t xw[2] = {xr.x ^ 0x80808080u, xr.y ^ 0x80808080u};
          float2 v[4];
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const float4 sx4 = ssx[pc * 2 + cc], sh4 = ssh[pc * 2 + cc];
            const float4 co4 = CORR ? sco[pc * 2 + cc] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int e2 = 0; e2 < 2; ++e2) {
              const int pp = cc * 4 + e2 * 2;
              const float2 sx2 = e2 ? make_float2(sx4.z, sx4.w) : make_float2(sx4.x, sx4.y);
              const float2 sh2 = e2 ? make_float2(sh4.z, sh4.w) : make_float2(sh4.x, sh4.y);
              const float2 co2 = e2 ? make_float2(co4.z, co4.w) : make_float2(co4.x, co4.y);
              const float2 xv = unpack2(xw[cc], e2 * 2);
              const float2 ao = make_float2((float)acc_o[pp], (float)acc_o[pp + 1]);
              const float2 ad = make_float2((float)acc_d[pp], (float)acc_d[pp + 1]);
              // y = s_x (s_M acc_diag + D x) + s_h (dec acc_off) + corr: five packed operations
              const float2 u2 = __ffma2_rn(sm2, ad, __fmul2_rn(Dh2, xv));
              const float2 r2 = __ffma2_rn(sx2, u2, co2);
              v[cc * 2 + e2] = __ffma2_rn(sh2, __fmul2_rn(dec2, ao), r2);
            }
            if (YT == 0)   // 4 values = one 16-byte chunk
              *reinterpret_cast<float4*>(srow + ((((pc & 3) * 2 + cc) ^ (lane & 7)) << 4)) =
                  make_float4(v[cc * 2].x, v[cc * 2].y, v[cc * 2 + 1].x, v[cc * 2 + 1].y);
          }
          if (YT != 0) {  // 8 values = one 16-byte chunk
            uint32_t h[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              if (YT == 1) {
                const __half2 hv = __floats2half2_rn(v[e].x, v[e].y);
                h[e] = *reinterpret_cast<const uint32_t*>(&hv);
              } else {
                const __nv_bfloat162 bv = __floats2bfloat162_rn(v[e].x, v[e].y);
                h[e] = *reinterpret_cast<const uint32_t*>(&bv);
              }
            }
            *reinterpret_cast<uint4*>(srow + ((pc ^ (lane & 7)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
          }
          if (TAPS && (a.taps.acc_off || a.taps.acc_diag)) {
            const i64 o = ((t.tok0 + ei) * d.H + t.h) * P + pc * 8;
#pragma unroll
            for (int pp = 0; pp < 8; ++pp) {
              if (a.taps.acc_off) a.taps.acc_off[o + pp] = acc_o[pp];
              if (a.taps.acc_diag) a.taps.acc_diag[o + pp] = acc_d[pp];
            }
          }
        }
        if ((pc & (PPR - 1)) == PPR - 1) {   // 128 bytes of every row are staged: store them
          if (pc == 7) tc_fence_before();
          fence_async_smem();
          __syncwarp();
          if (pc == 7 && lane < 3) {         // one release each, side by side
            mbar_arrive(&bars[lane == 0 ? B_ACC_FREE + a4 : lane == 1 ? B_X_FREE + xs : B_ROW_FREE + (n & 7)]);
          } else if (lane == 3 && q * 32 < TM) {
            tma_store_3d(&tm_y, ystage, (pc / PPR) * 32, t.h, (int)(t.tok0 + t.it * TM + q * 32));
            tma_store_commit();
          }
        }
      }
      if (ntpu == 2) {   // the same tile of the next head
        const int it = t.it;
        next_head(t, d, a.w, TM, ntpu);
        t.it = it;
        t.KJ = (it + 1) * TM;
      } else {
        next_tile(t, d, a.w, TM, ntpu);
        next_tile(t, d, a.w, TM, ntpu);
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

ssdi8_status_t launch_chunk_scan(const Dims& d, const int8_t* xq, const int8_t* Cq,
                                 const int8_t* CBq, const int8_t* hq, const float* s_x,
                                 const float* s_C, const float* s_cb, const float* s_h,
                                 const float* pack, const float* D,
                                 const float* corr, void* y, int ydt, int32_t* status, const ScanTaps& taps,
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
    const uint64_t eb = ydt ? 2 : 4;  // bytes per element of y
    uint64_t dims[3] = {(uint64_t)d.P, (uint64_t)d.H, T};
    uint64_t str[2] = {(uint64_t)d.P * eb, (uint64_t)d.H * d.P * eb};
    uint32_t box[3] = {ydt ? 64u : 32u, 1, 32};   // 128 bytes of a row per store
    if (!encode_tensor_map(&tm_y, y, (int)eb, 3, dims, str, box, 128)) return SSDI8_ERR_CUDA;
  }
  int dev = 0, sms = 0;
  SSDI8_CUDA_CHECK(cudaGetDevice(&dev));
  SSDI8_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  UnitWalk walk;
  int grid_i = 0;
  if (!make_unit_walk(d, TM, sms, &walk, &grid_i)) return SSDI8_ERR_SHAPE;
  ScanArgs a = {s_x, s_C, s_cb, s_h, pack, D, corr, static_cast<uint8_t*>(y), status, taps, d, walk};
  const size_t smem = SMEM_BYTES + 1024;
  const unsigned grid = (unsigned)grid_i;
  const bool tp = taps.acc_off || taps.rowmax || taps.Mq || taps.acc_diag;
  auto launch = [&](auto kernel) -> ssdi8_status_t {
    SSDI8_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    return launch_pdl(kernel, dim3(grid), dim3(kThreads), smem, st, tm_C, tm_h, tm_x, tm_cb, tm_y, a) == cudaSuccess ? SSDI8_OK : SSDI8_ERR_CUDA;
  };
  if (tp && ydt) return SSDI8_ERR_UNSUPPORTED;  // the taps come with binary32 y only
  const bool big = d.Q >= 128;
  auto pick = [&](auto corr_c, auto big_c) -> ssdi8_status_t {
    constexpr bool C = decltype(corr_c)::value, B = decltype(big_c)::value;
    if (tp) return launch(chunk_scan_tc<C, true, 0, B>);
    if (ydt == 0) return launch(chunk_scan_tc<C, false, 0, B>);
    if (ydt == 1) return launch(chunk_scan_tc<C, false, 1, B>);
    return launch(chunk_scan_tc<C, false, 2, B>);
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

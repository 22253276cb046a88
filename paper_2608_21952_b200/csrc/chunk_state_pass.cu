// ChunkState + StatePassing fused, chunk-sequential per (batch, head): the fp32 chunk-local
// state never goes to HBM.  For chunk k = 0 .. c-1 of one (b, h):
//   Xs_q[i,p]   = rne(fmul(fmul(float(xq[i,p]), fdiv(s_x, s_xs)), LUT_state[i]))       (Eq. 3)
//   acc_st[n,p] = sum_i Bq[i,n] Xs_q[i,p]            INT8 MMA over the chunk's tokens, INT32 in TMEM
//   loc[p,n]    = fmul(float(acc_st), fmul(s_xs[h,p], s_B[g]))                         (Eq. 4 rescale)
//   hq[k][p,n]  = rne(fmul(S[p,n], fdiv(1, s_h[h,p])))     (state entering chunk k, int8 for ChunkScan1)
//   S[p,n]      = fmaf(Gamma_k, S[p,n], loc[p,n])                                      (Eq. 6)
// and final_state = S after the last chunk.  The running state lives in registers: the
// accumulator has the state index n on the TMEM lanes, so thread (lane n) keeps S[., n] for its
// 32 channels p; the state itself is kept in tensor memory beside the accumulator (64 more columns,
// read and written 8 columns at a time), which leaves the threads with few registers so that three CTAs
// fit an SM: the kernel is a chain of short dependent steps per chunk, and what fills an SM is other
// CTAs' chains.  The xq tiles arrive by TMA double-buffered across chunks, the Bq tile of a chunk is
// single-buffered (requested when the MMAs of the chunk before have finished, needed only when the
// accumulator is free again); each re-quantisation
// warp owns whole 32-token slabs and issues their MMAs itself (the accumulator is opened by the warp
// that owns slab 0, the others order their MMAs after it through an mbarrier); hq leaves through
// a shared-memory tile and one TMA store per chunk.  Same arithmetic, operation for operation,
// as the separate kernels (chunk_state.cu, state_passing.cu).
// I8S = true selects the paper's own state format (Section 4.2, Eq. 4 and Eq. 7): the state is an
// int8 code with the one per-(H,P) scale s_h, the chunk-local state goes INT32 -> INT8 in
// registers, and the recurrence is integer with a fixed-point decay:
//   locq = rne(fmul(float(acc_st), fdiv(fmul(s_xs, s_B), s_h)));  Gq = rne(fmul(Gamma_k, 128))
//   Sq   = sat(locq + ((Gq * Sq + 64) >> 7));  hq[k] = Sq before the update;  final = fmul(float(Sq), s_h)
#include "kernels.h"
#include "sm100.cuh"

namespace ssdi8 {
namespace {

using namespace sm100;

struct FusedArgs {
  const float* s_x; const float* s_xs; const float* s_B; const float* s_h; const float* pack;
  const float* gamma; const float* init; float* final_state;
  float* tap_loc; float* tap_prev; int8_t* tap_Xsq; int32_t* tap_acc; int32_t* status;
  Dims d;
  int n_full;  // CTAs below this index own a whole (batch, head); the rest own one part of one
  int split;   // parts per (batch, head) of the rest: 2 (halves of 32 channels) or 4 (quarters of 16)
};

constexpr int kStateThreads = 256;   // warps 0-7: running state, hq, MMA issue, TMA
constexpr int kQuantThreads = 128;   // warps 8-11: Q(X_scaled) of the next chunk, one chunk ahead
constexpr int kThreads = kStateThreads + kQuantThreads;
constexpr uint32_t XSTAGE = 16384;                // xq rows [Q][64] of one chunk
constexpr uint32_t OFF_X = 0;                     // two stages
constexpr uint32_t OFF_B = 2 * XSTAGE;            // Bq rows [Q][N] of one chunk (single buffer)
constexpr uint32_t OFF_HQ = OFF_B + 32768;        // [64 p][N] int8 staging of hq
constexpr uint32_t OFF_LUT = OFF_HQ + 8192;       // 2 x [256] floats
constexpr uint32_t OFF_COL = OFF_LUT + 2048;      // [64] loc scale, [64] 1 / s_h, [64] s_h
constexpr uint32_t OFF_BAR = OFF_COL + 768;
constexpr uint32_t SMEM_BYTES = OFF_BAR + 64;     // 76 608 bytes: three CTAs per SM
constexpr uint32_t kTmemCols = 128;               // accumulator in columns 0..63, running state in 64..127

enum { B_XFULL = 0, B_BFULL = 2, B_OPEN = 3, B_MMA = 4, B_ACC_FREE = 5, B_COUNT = 6 };

__device__ __forceinline__ void named_bar(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// TAPS: any of the intermediate-tensor taps is requested (tests); the production instance carries no tap code
// NCQ: 16-channel chunks of the head this CTA owns (4 = the whole head, 1 = one quarter)
template <bool I8S, bool TAPS, int NCQ>
__device__ __forceinline__ void fused_body(const CUtensorMap& tm_B, const CUtensorMap& tm_x, const CUtensorMap& tm_hq,
                                           const FusedArgs& a, const int unit, const int c0) {
  // (no padding for the 1024-byte alignment the swizzled tiles need: three CTAs fill the SM's shared
  // memory to the last kilobyte; the launcher checks that the kernel uses no static shared memory, so
  // the dynamic part starts at the window's base, and the kernel checks the address itself)
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  constexpr int ncq = NCQ;
  uint8_t* smem = smem_raw;
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0 && a.status) atomicExch(a.status, (int32_t)SSDI8_ERR_ALIGN);
    return;
  }
  const Dims& d = a.d;
  const int Q = d.Q, N = d.N, P = d.P;
  const int TQ = Q < 128 ? Q : 128;  // rows per TMA box
  const int h = unit % d.H, b = unit / d.H;
  const int g = h / (d.H / d.G);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  uint8_t* sHQ = smem + OFF_HQ;
  float* col_scale = reinterpret_cast<float*>(smem + OFF_COL);
  float* col_invh = col_scale + 64;
  float* col_sh = col_invh + 64;
  const i64 bh = (i64)b * d.H + h;
  const i64 unit0 = bh * d.c;

  if (tid == 0) {
    mbar_init(&bars[B_XFULL], 1);
    mbar_init(&bars[B_XFULL + 1], 1);
    mbar_init(&bars[B_BFULL], 1);
    mbar_init(&bars[B_OPEN], 1);
    mbar_init(&bars[B_MMA], Q / 32 < kQuantThreads / 32 ? Q / 32 : kQuantThreads / 32);   // one commit per issuing warp
    mbar_init(&bars[B_ACC_FREE], kStateThreads / 32);
    fence_mbar_init();
    tma_prefetch_desc(&tm_B);
    tma_prefetch_desc(&tm_x);
    tma_prefetch_desc(&tm_hq);
  }
  if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
  pdl_wait();   // everything below reads global memory
  // (after the wait, not before it: ChunkBMM, launched next, reads and writes global memory without waiting
  // for this kernel, so it must not be scheduled before this kernel's predecessors have completed)
  pdl_launch_dependents();
  if (tid < 64) {
    const float sxb = __fmul_rn(a.s_xs[h * P + tid], a.s_B[g]), sh = a.s_h[h * P + tid];
    col_scale[tid] = I8S ? __fdiv_rn(sxb, sh) : sxb;
    col_invh[tid] = __fdiv_rn(1.0f, sh);
    col_sh[tid] = sh;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  auto issue_x = [&](int k) {  // thread 0 only: xq rows and LUT_state of chunk k
    const int s = k & 1;
    const i64 tok0 = (i64)b * d.L + (i64)k * Q;
    mbar_expect_tx(&bars[B_XFULL + s], (uint32_t)(Q * 64 + Q * 4));
    // LUT_state of the chunk arrives with the tile (a global load here would sit on the
    // re-quantisation group's critical path)
    bulk_load(smem + OFF_LUT + s * 1024, a.pack + ((unit0 + k) * kPackRows + PACK_LUT) * Q, (uint32_t)(Q * 4),
              &bars[B_XFULL + s]);
    for (int i0 = 0; i0 < Q; i0 += TQ)
      tma_load_3d(smem + OFF_X + s * XSTAGE + i0 * 64, &tm_x, &bars[B_XFULL + s], 0, h, (int)(tok0 + i0));
  };
  auto issue_B = [&](int k) {  // thread 0 only: Bq rows of chunk k, once the MMAs of chunk k-1 have finished
    const i64 tok0 = (i64)b * d.L + (i64)k * Q;
    mbar_expect_tx(&bars[B_BFULL], (uint32_t)(Q * N));
    for (int i0 = 0; i0 < Q; i0 += TQ)
      tma_load_3d(smem + OFF_B + i0 * N, &tm_B, &bars[B_BFULL], 0, g, (int)(tok0 + i0));
  };

  if (tid >= kStateThreads) {
    // ------------------------------------------------------------ Q(X_scaled), one chunk ahead of the state warps
    const int qt = tid - kStateThreads;
    constexpr int lq = ncq == 4 ? 2 : ncq == 2 ? 1 : 0;  // log2(chunks per row in this CTA's range)
    const int c = c0 + (qt & (ncq - 1));  // 16-byte chunk (16 channels) of every row this thread visits
    float rx[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const int hp = h * P + c * 16 + e;
      rx[e] = __fdiv_rn(a.s_x[hp], a.s_xs[hp]);
    }
    // Rows that re-quantise to zero (the sparsity Eq. 3 rests on: LUT_state decays towards the start
    // of a chunk).  fmul is monotone, so with rxm >= |rx| of every channel of this CTA's range,
    // fmul(fmul(127, rxm), |LUT_state[i]|) < 1/2 implies |fmul(fmul(x, rx), LUT_state[i])| < 1/2 for every
    // code x: row i of Q(X_scaled) is all zeros, exactly.  Such a row is stored as zeros without the
    // arithmetic, and a 32-token slab of such rows is left out altogether (no MMA).
    float rxm = 0.f;
#pragma unroll
    for (int e = 0; e < 16; ++e) rxm = fmaxf(rxm, fabsf(rx[e]));
    if (ncq >= 2) rxm = fmaxf(rxm, __shfl_xor_sync(0xffffffffu, rxm, 1));
    if (ncq == 4) rxm = fmaxf(rxm, __shfl_xor_sync(0xffffffffu, rxm, 2));
    const float b127 = __fmul_rn(127.0f, rxm);
#pragma unroll 1
    for (int k = 0; k < d.c; ++k) {
      const int s = k & 1;
      uint8_t* sX = smem + OFF_X + s * XSTAGE;
      float* lut = reinterpret_cast<float*>(smem + OFF_LUT) + s * 256;
      const i64 tok0 = (i64)b * d.L + (i64)k * Q;
      // one warp polls for the tiles; the others wait at a hardware barrier, which costs no issue slots
      if (qt < 32) mbar_wait_inline<256>(&bars[B_XFULL + s], (k >> 1) & 1, a.status);
      named_bar(2, kQuantThreads);
      // a warp owns whole 32-token slabs (slab = one MMA): rows of a slab are split over the lanes,
      // and the warp's lane 0 issues the slab's MMA as soon as the warp has re-quantised it, so no
      // warp waits for another.  The accumulator is opened by the MMA of the first live slab
      // (accumulate = 0); the other issuing threads order their first MMA of the chunk after it
      // through B_OPEN.  A chunk without a live slab opens with its last slab stored as zeros.
      const int qw = qt >> 5;
      const int nsl = Q / 32;
      uint32_t lm = 0;   // live slabs of the chunk (every warp computes the same mask)
      for (int sl = 0; sl < nsl; ++sl) {
        const bool dead = __fmul_rn(b127, fabsf(lut[sl * 32 + lane])) < 0.5f;
        if (!__all_sync(0xffffffffu, dead)) lm |= 1u << sl;
      }
      const bool zero_open = lm == 0;
      if (zero_open) lm = 1u << (nsl - 1);
      const int first = __ffs((int)lm) - 1;
      const uint32_t sBa = smem_u32(smem + OFF_B), sXa = smem_u32(sX);
      const uint32_t idesc = idesc_s8(N, 64, 1, 1);
      const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
      bool mine = false;   // this warp owns a live slab
#pragma unroll 1
      for (int sl = qw; sl < nsl; sl += kQuantThreads / 32) {
        if (!((lm >> sl) & 1u)) {
          if (TAPS && a.tap_Xsq) {
            for (int i = sl * 32 + (lane >> lq); i < sl * 32 + 32; i += 32 >> lq)
              *reinterpret_cast<uint4*>(a.tap_Xsq + ((tok0 + i) * d.H + h) * P + c * 16) = zero4;
          }
          continue;
        }
        mine = true;
#pragma unroll 1
        for (int i = sl * 32 + (lane >> lq); i < sl * 32 + 32; i += 32 >> lq) {
          uint4* ptr = reinterpret_cast<uint4*>(sX + swz_off((uint32_t)i, (uint32_t)c, 64));
          const float l = lut[i];
          if (zero_open || __fmul_rn(b127, fabsf(l)) < 0.5f) {
            *ptr = zero4;
            if (TAPS && a.tap_Xsq) *reinterpret_cast<uint4*>(a.tap_Xsq + ((tok0 + i) * d.H + h) * P + c * 16) = zero4;
            continue;
          }
          const uint4 w4 = *ptr;
          const uint32_t ww[4] = {w4.x ^ 0x80808080u, w4.y ^ 0x80808080u, w4.z ^ 0x80808080u, w4.w ^ 0x80808080u};
          const float2 l2 = make_float2(l, l);
          uint32_t o[4];
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            uint32_t q4[4];
#pragma unroll
            for (int e = 0; e < 4; e += 2) {
              const float2 xf = __fadd2_rn(
                  make_float2(__uint_as_float(__byte_perm(ww[w], 0x4B400000u, 0x7650u + e)),
                              __uint_as_float(__byte_perm(ww[w], 0x4B400000u, 0x7651u + e))),
                  make_float2(-kMagicIn, -kMagicIn));
              const uint2 c2 = rne_clamp_bits2(__fmul2_rn(__fmul2_rn(xf, make_float2(rx[w * 4 + e], rx[w * 4 + e + 1])), l2));
              q4[e] = c2.x;
              q4[e + 1] = c2.y;
            }
            o[w] = pack4_bits(q4[0], q4[1], q4[2], q4[3]);
          }
          const uint4 v = make_uint4(o[0], o[1], o[2], o[3]);
          *ptr = v;
          if (TAPS && a.tap_Xsq) *reinterpret_cast<uint4*>(a.tap_Xsq + ((tok0 + i) * d.H + h) * P + c * 16) = v;
        }
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0 && qw < nsl) {
        if (mine) {
          if ((first & (kQuantThreads / 32 - 1)) == qw) {
            mbar_wait_inline<0>(&bars[B_ACC_FREE], (k & 1) ^ 1, a.status);   // the state warps have read chunk k-1
          } else {
            mbar_wait_inline<0>(&bars[B_OPEN], k & 1, a.status);
          }
          mbar_wait_inline<0>(&bars[B_BFULL], k & 1, a.status);   // the chunk's Bq rows have landed
          tc_fence_after();
#pragma unroll 1
          for (int sl = qw; sl < nsl; sl += kQuantThreads / 32) {
            if (!((lm >> sl) & 1u)) continue;
            mma_s8_ss(tmem, tile_desc(sBa + 32 * sl * N, (uint32_t)N), tile_desc(sXa + 32 * sl * 64, 64), idesc, sl != first);
            if (sl == first) {
              tc_fence_before();
              mbar_arrive(&bars[B_OPEN]);
            }
          }
        }
        mma_commit(&bars[B_MMA]);   // arrives when this thread's MMAs are done (at once if it issued none)
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------ state warps
    // M = 128: accumulator row n on TMEM lane n; M = 64: row n on lane (n % 16) + 32 (n / 16),
    // i.e. the first 16 lanes of each warp's quarter
    const int q = warp & 3, ch = warp >> 2;
    constexpr int npp = 8 * ncq;             // channels per thread
    const int cb = 16 * c0 + ch * npp;       // first channel of this thread
    const bool ok = (N == 128) || (lane < 16);
    const int n = (N == 128) ? q * 32 + lane : q * 16 + lane;
    // the running state S[p, n]: fp32, or (I8S) the integer code, in tensor-memory columns 64 + p of lane n
    const uint32_t tlane = tmem + ((uint32_t)(q * 32) << 16);
    const uint32_t tS = tlane + 64u + (uint32_t)cb;
#pragma unroll
    for (int p0 = 0; p0 < 32; p0 += 8) {
      if (p0 < npp) {
        int sv[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float v = (a.init && ok) ? a.init[(bh * P + cb + p0 + e) * N + n] : 0.f;
          sv[e] = I8S ? (int)(int8_t)(rne_clamp_bits(__fmul_rn(v, col_invh[(cb + p0 + e) & 63])) & 0xffu) : __float_as_int(v);
        }
        tmem_st8(tS + (uint32_t)p0, sv);
      }
    }
    tmem_st_wait();
    if (tid == 0) {
      issue_x(0);
      issue_B(0);
      if (d.c > 1) issue_x(1);
    }
#pragma unroll 1
    for (int k = 0; k < d.c; ++k) {
      const float gam = a.gamma[unit0 + k];
      if (tid == 0 && k > 0) tma_store_wait_read();  // last chunk's hq store has read the staging tile
      named_bar(1, kStateThreads);  // also: every state thread has read the accumulator of chunk k-1
      // ---- hq[k] = codes of the state entering this chunk (and the prev tap).  They are formed here, ahead
      // of the wait for the chunk's MMAs, from a second read of the state; forming them in the update pass of
      // the chunk before, while the new values are in registers, puts them behind that wait on the chain of
      // the chunk and was measured slower (0.0568 against 0.0536 ms at batch 8 x 2048 x 80 heads).
      {
        const i64 obase = (((((i64)b * d.c + k) * d.H + h) * P) + cb) * N + n;
        // batches of 8: all loads of a batch before its byte stores (a byte store may alias anything,
        // so interleaving them would serialise the loop on shared-memory latency).  The tensor-memory
        // loads are warp-wide; lanes without a state row (N = 64) skip what follows them.
#pragma unroll
        for (int p0 = 0; p0 < 32; p0 += 8) {
          if (p0 < npp) {
            int sv[8];
            tmem_ld8(tS + (uint32_t)p0, sv);
            tmem_ld_wait();
            if (ok) {
              uint32_t code[8];
              // (cb is a multiple of 8: the eight reciprocals are two 16-byte loads)
              const float4 i0 = *reinterpret_cast<const float4*>(col_invh + cb + p0);
              const float4 i1 = *reinterpret_cast<const float4*>(col_invh + cb + p0 + 4);
              const float ih[8] = {i0.x, i0.y, i0.z, i0.w, i1.x, i1.y, i1.z, i1.w};
#pragma unroll
              for (int e = 0; e < 8; e += 2) {
                if (I8S) {
                  code[e] = (uint32_t)sv[e];
                  code[e + 1] = (uint32_t)sv[e + 1];
                } else {
                  const uint2 c2 = rne_clamp_bits2(__fmul2_rn(make_float2(__int_as_float(sv[e]), __int_as_float(sv[e + 1])),
                                                              make_float2(ih[e], ih[e + 1])));
                  code[e] = c2.x;
                  code[e + 1] = c2.y;
                }
              }
              uint8_t* hrow = sHQ + (cb + p0) * N + n;
#pragma unroll
              for (int e = 0; e < 8; ++e, hrow += N) *hrow = (uint8_t)code[e];
              if (TAPS && !I8S && a.tap_prev) {
#pragma unroll
                for (int e = 0; e < 8; ++e) a.tap_prev[obase + (i64)(p0 + e) * N] = __int_as_float(sv[e]);
              }
            }
          }
        }
      }
      fence_async_smem();
      // one warp polls for the MMAs of this chunk; the barrier passes their completion on to the others
      if (warp == 0) mbar_wait_inline<256>(&bars[B_MMA], k & 1, a.status);
      named_bar(1, kStateThreads);
      // ---- hq[k] leaves by TMA
      if (tid == 0) {
        for (int j = c0; j < c0 + ncq; ++j)  // 16 channels (rows of hq) per store
          tma_store_2d(&tm_hq, sHQ + 16 * j * N, 0, (int)(((((i64)b * d.c + k) * d.H + h) * P) + 16 * j));
        tma_store_commit();
      }
      // ---- epilogue of the MMA: S = fmaf(Gamma_k, S, loc), 8 channels at a time
      tc_fence_after();
      if (tid == 0) {   // the MMAs of chunk k have finished reading the Bq buffer and xq stage s
        if (k + 1 < d.c) issue_B(k + 1);
        if (k + 2 < d.c) issue_x(k + 2);
      }
#pragma unroll
      for (int hf = 0; hf < 4; ++hf) {       // 8 channels at a time
        if (hf < ncq) {
        int acc[8], sv[8];
        tmem_ld8(tlane + (uint32_t)(cb + hf * 8), acc);
        tmem_ld8(tS + (uint32_t)(hf * 8), sv);
        tmem_ld_wait();
        if (ok) {
          const i64 obase = (((((i64)b * d.c + k) * d.H + h) * P) + cb + hf * 8) * N + n;
          const float4 c0v = *reinterpret_cast<const float4*>(col_scale + cb + hf * 8);
          const float4 c1v = *reinterpret_cast<const float4*>(col_scale + cb + hf * 8 + 4);
          const float cscale[8] = {c0v.x, c0v.y, c0v.z, c0v.w, c1v.x, c1v.y, c1v.z, c1v.w};
#pragma unroll
          for (int e = 0; e < 8; e += 2) {
            const float2 af = __fadd2_rn(make_float2(__int_as_float(acc[e] + 0x4B400000), __int_as_float(acc[e + 1] + 0x4B400000)),
                                         make_float2(-kMagicOut, -kMagicOut));   // exact for |acc| < 2^22
            const float2 l2 = __fmul2_rn(af, make_float2(cscale[e], cscale[e + 1]));
            if (TAPS && a.tap_acc) {
              a.tap_acc[obase + (i64)e * N] = acc[e];
              a.tap_acc[obase + (i64)(e + 1) * N] = acc[e + 1];
            }
            if (I8S) {
              const int Gq = __float2int_rn(__fmul_rn(gam, 128.0f));
#pragma unroll
              for (int j = 0; j < 2; ++j) {
                const int locq = (int)(int8_t)(rne_clamp_bits(j ? l2.y : l2.x) & 0xffu);
                const int Sn = locq + ((Gq * sv[e + j] + 64) >> 7);
                sv[e + j] = max(-127, min(127, Sn));
              }
            } else {
              if (TAPS && a.tap_loc) {
                a.tap_loc[obase + (i64)e * N] = l2.x;
                a.tap_loc[obase + (i64)(e + 1) * N] = l2.y;
              }
              const float2 s2 = __ffma2_rn(make_float2(gam, gam),
                                           make_float2(__int_as_float(sv[e]), __int_as_float(sv[e + 1])), l2);
              sv[e] = __float_as_int(s2.x);
              sv[e + 1] = __float_as_int(s2.y);
            }
          }
        }
        tmem_st8(tS + (uint32_t)(hf * 8), sv);
      }
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars[B_ACC_FREE]);  // this warp has read the accumulator of chunk k
    }
    if (a.final_state) {
#pragma unroll
      for (int p0 = 0; p0 < 32; p0 += 8) {
        if (p0 < npp) {
          int sv[8];
          tmem_ld8(tS + (uint32_t)p0, sv);
          tmem_ld_wait();
          if (ok) {
#pragma unroll
            for (int e = 0; e < 8; ++e)
              a.final_state[(bh * P + cb + p0 + e) * N + n] =
                  I8S ? __fmul_rn((float)sv[e], col_sh[cb + p0 + e]) : __int_as_float(sv[e]);
          }
        }
      }
    }
    if (tid == 0) tma_store_wait_read();
  }
  drain_after_timeout(a.status);
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

// Column range of a CTA: 16-channel chunks c0 .. c0 + ncq - 1 of one head.  Whole heads first, then
// the heads of a nearly empty last wave, split in halves or quarters so that they spread over the
// free slots (operand tiles and the MMA stay full width: only the re-quantisation, the state
// update and the hq rows are restricted to the range).
template <bool I8S, bool TAPS>
__global__ void __launch_bounds__(kThreads, 3)
chunk_state_pass_tc(const __grid_constant__ CUtensorMap tm_B, const __grid_constant__ CUtensorMap tm_x,
                    const __grid_constant__ CUtensorMap tm_hq, const FusedArgs a) {
  if ((int)blockIdx.x < a.n_full) {
    fused_body<I8S, TAPS, 4>(tm_B, tm_x, tm_hq, a, (int)blockIdx.x, 0);
  } else if (a.split == 2) {
    const int r = (int)blockIdx.x - a.n_full;
    fused_body<I8S, TAPS, 2>(tm_B, tm_x, tm_hq, a, a.n_full + (r >> 1), 2 * (r & 1));
  } else {
    const int r = (int)blockIdx.x - a.n_full;
    fused_body<I8S, TAPS, 1>(tm_B, tm_x, tm_hq, a, a.n_full + (r >> 2), r & 3);
  }
}

}  // namespace

ssdi8_status_t launch_chunk_state_passing(const Dims& d, const int8_t* xq, const int8_t* Bq,
                                          const float* s_x, const float* s_xs, const float* s_B,
                                          const float* s_h, const float* pack, const float* gamma,
                                          const float* init, int8_t* hq, float* final_state,
                                          float* tap_loc, float* tap_prev, int8_t* tap_Xsq,
                                          int32_t* tap_acc, int32_t* status, bool int8_state,
                                          cudaStream_t st) {
  const int TQ = d.Q < 128 ? d.Q : 128;
  const uint64_t T = (uint64_t)d.b * d.L;
  CUtensorMap tm_B, tm_x, tm_hq;
  {
    uint64_t dims[3] = {(uint64_t)d.N, (uint64_t)d.G, T};
    uint64_t str[2] = {(uint64_t)d.N, (uint64_t)d.G * d.N};
    uint32_t box[3] = {(uint32_t)d.N, 1, (uint32_t)TQ};
    if (!encode_tensor_map(&tm_B, Bq, 1, 3, dims, str, box, d.N)) return SSDI8_ERR_CUDA;
  }
  {
    uint64_t dims[3] = {(uint64_t)d.P, (uint64_t)d.H, T};
    uint64_t str[2] = {(uint64_t)d.P, (uint64_t)d.H * d.P};
    uint32_t box[3] = {64, 1, (uint32_t)TQ};
    if (!encode_tensor_map(&tm_x, xq, 1, 3, dims, str, box, 64)) return SSDI8_ERR_CUDA;
  }
  {
    uint64_t dims[2] = {(uint64_t)d.N, (uint64_t)d.b * d.c * d.H * d.P};
    uint64_t str[1] = {(uint64_t)d.N};
    uint32_t box[2] = {(uint32_t)d.N, 16};
    if (!encode_tensor_map(&tm_hq, hq, 1, 2, dims, str, box, 0)) return SSDI8_ERR_CUDA;
  }
  // (batch, head) units over the CTA slots of the device (3 CTAs per SM): whole waves of whole
  // units, and the units of a last, partly filled wave as four quarter-width CTAs each, which pack
  // into that wave's free slots (a quarter costs about a third of a whole unit: the operand tiles
  // and the MMA stay full width)
  int dev = 0, sms = 0;
  SSDI8_CUDA_CHECK(cudaGetDevice(&dev));
  SSDI8_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int units = d.H * d.b, slots = 3 * sms;
  // Whole (batch, head) units wherever the device is filled: with three CTAs per SM the kernel is bound
  // by instruction issue, so a partly filled last wave of whole units runs faster per CTA and costs less
  // than the same units cut into more CTAs (measured at 640 units on 444 slots: 0.054 ms whole, 0.056 ms
  // in halves, 0.067 ms in quarters).  Only a workload that leaves most slots empty (fewer units than an
  // eighth of a wave beyond the full waves) is cut into quarter-width CTAs, which spreads it over more
  // SMs (24 units: 0.0225 ms in quarters against 0.0265 ms whole).
  int n_full = units / slots * slots;
  int split = 4;
  if (8 * (units - n_full) > slots) n_full = units;
  FusedArgs a = {s_x, s_xs, s_B, s_h, pack, gamma, init, final_state, tap_loc, tap_prev, tap_Xsq, tap_acc,
                 status, d, n_full, split};
  const size_t smem = SMEM_BYTES;
  const unsigned grid = (unsigned)(n_full + split * (units - n_full));
  const bool taps = tap_loc || tap_prev || tap_Xsq || tap_acc;
  auto launch = [&](auto kernel) -> ssdi8_status_t {
    cudaFuncAttributes fa;
    SSDI8_CUDA_CHECK(cudaFuncGetAttributes(&fa, kernel));
    if (fa.sharedSizeBytes != 0) return SSDI8_ERR_CUDA;   // the dynamic part must start at the window's base
    SSDI8_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    return launch_pdl(kernel, dim3(grid), dim3(kThreads), smem, st, tm_B, tm_x, tm_hq, a) == cudaSuccess ? SSDI8_OK : SSDI8_ERR_CUDA;
  };
  ssdi8_status_t ls;
  if (int8_state)
    ls = taps ? launch(chunk_state_pass_tc<true, true>) : launch(chunk_state_pass_tc<true, false>);
  else
    ls = taps ? launch(chunk_state_pass_tc<false, true>) : launch(chunk_state_pass_tc<false, false>);
  if (ls != SSDI8_OK) return ls;
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

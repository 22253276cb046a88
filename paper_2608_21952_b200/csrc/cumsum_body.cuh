// ChunkCumsum (Algorithm 2, module 1) and the per-token scalars every later module derives
// from it.  For each (batch, head, chunk) it writes one contiguous pack of 6 rows of Q floats:
//   row 0  cs[i]    = (float) sum_{i'<=i} (double)dt (double)A_h, in token order   (dA_cs)
//   row 1  dt[i]
//   row 2  woff[i]  = fmul(dt_i, exp32(fsub(cs_ie, cs_i))), ie = last token of i's 16-token sub-block
//   row 3  atok[i]  = exp32(fsub(cs_i, cs_{i-1}))  (1 for i = 0): the per-token decay
//   row 4  bounds that let the scan kernel skip sub-blocks that cannot matter (they decide no
//          output bit): [c] = fmul(127, wmax_c), wmax_c the maximum of |woff| over the 16-token
//          sub-block c; [16 + c] = the maximum of the former over sub-blocks 0..c, times
//          1.00001, or +inf when cs is not non-increasing over the chunk (some dt A > 0), which
//          switches the early exits of the scan kernel off; [32 + I (I - 1) / 2 + c], c < I: the decay
//          between the ends of sub-blocks c and I - 1, exp32(fsub(cs[16 I - 1], cs[16 c + 15])), which
//          the scan kernel multiplies by a row's own decay to the end of sub-block I - 1; the rest of
//          the row is not written
//   row 5  lut[i]   = fmul(dt_i, exp32(fsub(cs_last, cs_i)))                       (LUT_state)
// and Gamma[b,h,k] = exp32(cs[Q-1]) (Decay_pass, Eq. 5).  The sum order is part of the definition
// (it decides rounding downstream), so each (b, chunk, head) is scanned sequentially by one
// thread: a block takes 8 heads x KC chunks, i.e. 8 KC sequential scans side by side (KC = 4 fills
// the 32 lanes of the scanning warp).  Loads and stores go through shared memory so that the
// [b,L,H] reads and the row writes coalesce.  Later kernels fetch a pack with one bulk copy and
// need no exponentials per token.
#pragma once
#include "kernels.h"

namespace ssdi8 {

constexpr int kCumsumHeads = 8;  // heads per block

// shared memory of a block: dt and cs rows of its 8 KC (head, chunk) units, their flags and bounds, and the
// binary64 increments dt A of the scan
__host__ __device__ inline size_t cumsum_smem_bytes(int Q, int KC, bool pre = false) {
  return sizeof(float) * (size_t)(kCumsumHeads * KC) * (2 * (size_t)(Q + 1) + 16 + (pre ? 2 * (size_t)Q + 2 : 0));
}

// One block's work: heads 8 bx .. and chunks KC kx .. of batch element b.  Any whole number of warps
// may run it (every loop strides by the block size); `tile` is cumsum_smem_bytes(Q, KC) of shared memory.
// SOFTPLUS: dt holds the raw time step and dt = softplus(dt + dt_bias[h]) (dt_bias may be NULL)
// is applied as the values are staged (Algorithm 2 module 1 starts there).
// (a template parameter: the binary64 softplus costs registers, and the plain instance must keep its occupancy)
// PRE: the scan's binary64 increments dt A are formed by all threads while dt is staged and kept in shared
// memory, which leaves the sequential part one addition per token.  That shortens a block's chain (what a
// small grid waits for: 0.0164 against 0.0184 ms at 2048 x 24 heads) and costs shared memory and binary64 work
// that a full device has no room for (0.027 against 0.025 ms at batch 8 x 2048 x 80 heads), so the launcher
// takes it for grids that leave SMs empty only; `tile` is then cumsum_smem_bytes(Q, KC, true).
template <int KC, bool SOFTPLUS = false, bool PRE = false>
__device__ __forceinline__ void cumsum_body(const float* __restrict__ dt, const float* __restrict__ A,
                                            float* __restrict__ pack, float* __restrict__ gamma,
                                            float* __restrict__ tap_cs, const Dims& d, int bx, int kx, int b,
                                            float* tile, const float* __restrict__ dt_bias = nullptr) {
  constexpr int CH = kCumsumHeads, NU = CH * KC;   // unit u = hh * KC + kk
  const int Q = d.Q, ld = Q + 1;
  const int lq = 31 - __clz(Q);  // Q is a power of two
  float* dts = tile;                   // [NU][Q + 1]; entry Q of a row: 1 if cs is non-increasing over the chunk
  float* css = tile + NU * ld;         // [NU][Q + 1]
  float* wmx = tile + 2 * NU * ld;     // [NU][16]: 127 max|woff| per 16-token sub-block
  // [NU][Q] binary64 increments (double)dt (double)A, exact; 8-byte aligned: 2 NU (Q + 1) + 16 NU floats precede it
  double* inc = reinterpret_cast<double*>(tile + 2 * NU * ld + 16 * NU);
  const int h0 = bx * CH, k0 = kx * KC;
  const int nh = min(CH, d.H - h0), nk = min(KC, d.c - k0);
  const i64 t0 = (i64)b * d.L + (i64)k0 * Q;
  const int ntok = nk * Q;             // tokens of the block's chunks (contiguous in time)
  // entry Q of a dt row: 1 until a token is met whose increment dt A is positive
  if (PRE) {
    if (threadIdx.x < NU) dts[threadIdx.x * ld + Q] = 1.0f;
    __syncthreads();
  }
  // (all loads of a round of 8 before the first store: the loads are the latency of this phase)
  for (int e0 = threadIdx.x; e0 < ntok * CH; e0 += 8 * blockDim.x) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + u * blockDim.x;
      const int t = e / CH, hh = e % CH;
      v[u] = (e < ntok * CH && hh < nh) ? __ldg(dt + (t0 + t) * d.H + h0 + hh) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + u * blockDim.x;
      const int t = e / CH, hh = e % CH;
      if (e < ntok * CH && hh < nh) {
        const float dv = SOFTPLUS ? softplus_dt(v[u], dt_bias ? __ldg(dt_bias + h0 + hh) : 0.f) : v[u];
        const float af = PRE ? __ldg(A + h0 + hh) : 0.f;
        const int un = hh * KC + (t >> lq), i = t & (Q - 1);
        dts[un * ld + i] = dv;
        // the scan's increment, formed here by all threads: the product of two binary32 numbers is exact in
        // binary64, so only the additions are left to the sequential part
        if (PRE) {
          inc[un * Q + i] = (double)dv * (double)af;
          if ((af > 0.f && dv > 0.f) || (af < 0.f && dv < 0.f)) dts[un * ld + Q] = 0.0f;
        }
      }
    }
  }
  __syncthreads();
  if (threadIdx.x < NU) {
    const int u = threadIdx.x, hh = u / KC, kk = u % KC;
    if (hh < nh && kk < nk) {
      double acc = 0.0;
      float last = 0.f;
      if (PRE) {
        // Q is a multiple of 8: the loads of 8 increments are independent, only the additions form the chain
        for (int i0 = 0; i0 < Q; i0 += 8) {
          double pr[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) pr[j] = inc[u * Q + i0 + j];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            acc += pr[j];
            last = (float)acc;
            css[u * ld + i0 + j] = last;
          }
        }
      } else {
        const double a = (double)A[h0 + hh];
        float dmin = 0.f, dmax = 0.f;  // every increment dt A <= 0  <=>  no dt has the sign of A
        // loads and products (exact in binary64) of 8 tokens are independent, only the additions form the chain
        for (int i0 = 0; i0 < Q; i0 += 8) {
          float dv[8];
          double pr[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            dv[j] = dts[u * ld + i0 + j];
            pr[j] = (double)dv[j] * a;
            dmin = fminf(dmin, dv[j]);
            dmax = fmaxf(dmax, dv[j]);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            acc += pr[j];
            last = (float)acc;
            css[u * ld + i0 + j] = last;
          }
        }
        const bool mono = a > 0.0 ? dmax <= 0.f : (a < 0.0 ? dmin >= 0.f : true);
        dts[u * ld + Q] = mono ? 1.0f : 0.0f;
      }
      gamma[((i64)b * d.H + h0 + hh) * d.c + k0 + kk] = exp32(last);
    }
  }
  __syncthreads();
  const uint64_t pol = l2_policy_evict_last();
  // per-token rows of the pack.  Consecutive threads take consecutive tokens of one unit, so a row's
  // stores coalesce and the 16 tokens of a sub-block sit in 16 adjacent lanes (Q is a multiple of 32)
  for (int e = threadIdx.x; e < NU * Q; e += blockDim.x) {
    const int u = e >> lq, i = e & (Q - 1);
    const int hh = u / KC, kk = u % KC;
    const bool live = hh < nh && kk < nk;    // (uniform over a warp: a warp stays inside one unit)
    float wo = 0.f;
    if (live) {
      const float* c = css + u * ld;
      const float ci = c[i], di = dts[u * ld + i];
      const i64 un = ((i64)b * d.H + h0 + hh) * d.c + k0 + kk;
      float* p = pack + ((un * kPackRows) << lq) + i;
      // (the pack is read by the state kernel and by ChunkScan after the quantisers and the state kernel have
      // streamed several times the size of L2: its lines are kept ahead of theirs)
      st_global_hint(p, ci, pol);
      st_global_hint(p + Q, di, pol);
      wo = __fmul_rn(di, exp32(__fsub_rn(c[i | 15], ci)));
      st_global_hint(p + PACK_WOFF * Q, wo, pol);
      st_global_hint(p + PACK_ATOK * Q, i > 0 ? exp32(__fsub_rn(ci, c[i - 1])) : 1.0f, pol);
      st_global_hint(p + PACK_LUT * Q, __fmul_rn(di, exp32(__fsub_rn(c[Q - 1], ci))), pol);
      if (tap_cs) tap_cs[(un << lq) + i] = ci;
    }
    // sub-block maxima of |woff|, times 127
    float m = fabsf(wo);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (live && (i & 15) == 0) wmx[u * 16 + (i >> 4)] = __fmul_rn(127.0f, m);
  }
  // block-to-block decays G[I][c], c < I (triangular: 120 entries for 16 sub-blocks); they need cs only,
  // so they go out ahead of the barrier that the bounds wait for
  const int nsb = Q >> 4, ntri = nsb * (nsb - 1) / 2;
  for (int e = threadIdx.x; e < NU * 128; e += blockDim.x) {
    const int u = e >> 7, idx = e & 127;
    const int hh = u / KC, kk = u % KC;
    if (hh >= nh || kk >= nk || idx >= ntri) continue;
    // I (I - 1) / 2 <= idx < (I + 1) I / 2; 1 + 8 idx is (2 I - 1)^2 at the lower end, so the root is exact there
    const int I = (int)((1.0f + sqrtf((float)(1 + 8 * idx))) * 0.5f);
    const int c = idx - I * (I - 1) / 2;
    const float* cc = css + u * ld;
    const i64 un = ((i64)b * d.H + h0 + hh) * d.c + k0 + kk;
    pack[((un * kPackRows + PACK_WMAX) << lq) + 32 + idx] = exp32(__fsub_rn(cc[16 * I - 1], cc[16 * c + 15]));
  }
  __syncthreads();
  for (int e = threadIdx.x; e < 32 * NU; e += blockDim.x) {   // the first 32 entries of the bounds row
    const int u = e >> 5, i = e & 31;
    const int hh = u / KC, kk = u % KC;
    if (hh >= nh || kk >= nk) continue;
    float m = 0.f;
    if (i < Q / 16) {
      m = wmx[u * 16 + i];
    } else if (i >= 16 && i < 16 + Q / 16) {
      for (int c = 0; c <= i - 16; ++c) m = fmaxf(m, wmx[u * 16 + c]);
      m = dts[u * ld + Q] != 0.f ? __fmul_rn(m, 1.00001f) : __int_as_float(0x7f800000);
    }
    const i64 un = ((i64)b * d.H + h0 + hh) * d.c + k0 + kk;
    pack[((un * kPackRows + PACK_WMAX) << lq) + i] = m;
  }
}

}  // namespace ssdi8

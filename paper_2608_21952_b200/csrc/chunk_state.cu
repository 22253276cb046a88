// ChunkState with the sparse-aware reformulation (Eq. 3) and the INT32 rescale (Eq. 4) on
// tcgen05 tensor cores.  One CTA per (batch, chunk, head):
//   LUT_state[i] = fmul(dt_i, exp32(fsub(cs_last, cs_i)))        (row 4 of the ChunkCumsum pack)
//   Xs_q[i,p]    = rne(fmul(fmul(float(xq[i,p]), fdiv(s_x, s_xs)), LUT_state[i]))   in place in smem
//   acc_st[n,p]  = sum_i Bq[i,n] Xs_q[i,p]     INT8 MMA over the tokens of the chunk, INT32 in TMEM
//   loc[p,n]     = fmul(float(acc_st), fmul(s_xs[h,p], s_B[g]))
// Both operands are token-major in HBM, i.e. MN-major for this contraction: TMA stages them
// as they are and the MMA reads them through MN-major descriptors (no transposes anywhere).
// The accumulator is held with the state index n on the TMEM lanes, so that each warp store
// of the epilogue writes 32 consecutive n of one p: full 128-byte lines of loc[p][n].
#include "kernels.h"
#include "sm100.cuh"

namespace ssdi8 {
namespace {

using namespace sm100;

struct StateArgs {
  const float* s_x; const float* s_xs; const float* s_B; const float* pack;
  float* loc; int8_t* tap_Xsq; int32_t* tap_acc; uint32_t* absmax_xs; int32_t* status;
  Dims d;
};

constexpr int kThreads = 256;
constexpr uint32_t OFF_B = 0;        // [Q][N]  Bq rows (token-major)
constexpr uint32_t OFF_X = 32768;    // [Q][64] xq rows -> Xs_q in place
constexpr uint32_t OFF_F = 49152;    // lut[256], bars, tmem slot
constexpr uint32_t SMEM_BYTES = OFF_F + 256 * 4 + 64;

__global__ void __launch_bounds__(kThreads, 3)
chunk_state_tc(const __grid_constant__ CUtensorMap tm_B, const __grid_constant__ CUtensorMap tm_x,
               const StateArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const Dims& d = a.d;
  const int Q = d.Q, N = d.N, P = d.P;
  const int TQ = Q < 128 ? Q : 128;  // rows per TMA box
  const int h = blockIdx.x, k = blockIdx.y, b = blockIdx.z;
  const int g = h / (d.H / d.G);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const i64 tok0 = (i64)b * d.L + (i64)k * Q;
  uint8_t* sB = smem + OFF_B;
  uint8_t* sX = smem + OFF_X;
  float* lut = reinterpret_cast<float*>(smem + OFF_F);
  uint64_t* bars = reinterpret_cast<uint64_t*>(lut + 256);  // [0] operands landed, [1] MMA done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
  const bool calib = a.absmax_xs != nullptr;

  if (tid == 0) {
    mbar_init(&bars[0], 1);
    mbar_init(&bars[1], 1);
    fence_mbar_init();
    tma_prefetch_desc(&tm_B);
    tma_prefetch_desc(&tm_x);
  }
  if (warp == 1 && !calib) tmem_alloc(tmem_slot, 64);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {
    mbar_expect_tx(&bars[0], (uint32_t)(Q * 64 + (calib ? 0 : Q * N)));
    for (int i0 = 0; i0 < Q; i0 += TQ) {
      tma_load_3d(sX + i0 * 64, &tm_x, &bars[0], 0, h, (int)(tok0 + i0));
      if (!calib) tma_load_3d(sB + i0 * N, &tm_B, &bars[0], 0, g, (int)(tok0 + i0));
    }
  }
  if (tid < Q) lut[tid] = a.pack[((((i64)b * d.H + h) * d.c + k) * kPackRows + PACK_LUT) * Q + tid];
  // per-column factors of this thread's 16 channels (16-byte chunk c of every row it visits)
  const int c = tid & 3;
  float rx[16];
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    const int hp = h * P + c * 16 + e;
    rx[e] = calib ? a.s_x[hp] : __fdiv_rn(a.s_x[hp], a.s_xs[hp]);
  }
  __syncthreads();
  mbar_wait(&bars[0], 0, a.status);

  // ---- X_scaled, re-quantised in place (thread: chunk c of rows tid/4, tid/4 + 64, ...)
  float mx[16];
#pragma unroll
  for (int e = 0; e < 16; ++e) mx[e] = 0.f;
  for (int i = tid >> 2; i < Q; i += kThreads / 4) {
    uint4* ptr = reinterpret_cast<uint4*>(sX + swz_off((uint32_t)i, (uint32_t)c, 64));
    const uint4 w4 = *ptr;
    const uint32_t ww[4] = {w4.x ^ 0x80808080u, w4.y ^ 0x80808080u, w4.z ^ 0x80808080u, w4.w ^ 0x80808080u};
    const float l = lut[i];
    if (calib) {
#pragma unroll
      for (int e = 0; e < 16; ++e)
        mx[e] = fmaxf(mx[e], fabsf(__fmul_rn(__fmul_rn(s8_to_f32(ww[e >> 2], e & 3), rx[e]), l)));
    } else {
      uint32_t o[4];
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        uint32_t q4[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
          q4[e] = rne_clamp_bits(__fmul_rn(__fmul_rn(s8_to_f32(ww[w], e), rx[w * 4 + e]), l));
        o[w] = pack4_bits(q4[0], q4[1], q4[2], q4[3]);
      }
      const uint4 v = make_uint4(o[0], o[1], o[2], o[3]);
      *ptr = v;
      if (a.tap_Xsq) *reinterpret_cast<uint4*>(a.tap_Xsq + ((tok0 + i) * d.H + h) * P + c * 16) = v;
    }
  }
  if (calib) {
#pragma unroll
    for (int e = 0; e < 16; ++e) atomicMax(a.absmax_xs + h * P + c * 16 + e, __float_as_uint(mx[e]));
    return;
  }
  fence_async_smem();
  __syncthreads();

  // ---- acc[n][p] = sum_i Bq[i][n] Xs_q[i][p]: A = Bq (MN-major, M = N states), B = Xs_q (MN-major)
  const uint32_t tmem = *tmem_slot;
  if (tid == 0) {
    tc_fence_after();
    const uint32_t idesc = idesc_s8(N, 64, 1, 1);
    for (int s = 0; s < Q / 32; ++s)
      mma_s8_ss(tmem, tile_desc(smem_u32(sB) + 32 * s * N, (uint32_t)N),
                tile_desc(smem_u32(sX) + 32 * s * 64, 64), idesc, s > 0);
    mma_commit(&bars[1]);
  }
  __syncwarp();
  mbar_wait(&bars[1], 0, a.status);
  tc_fence_after();

  // ---- epilogue.  M = 128: accumulator row n on TMEM lane n.  M = 64: row n on lane
  // (n % 16) + 32 (n / 16), i.e. the first 16 lanes of each warp's quarter.
  {
    const int q = warp & 3, ch = warp >> 2;
    int acc[32];
    tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(ch * 32), acc);
    tmem_ld_wait();
    const bool ok = (N == 128) || (lane < 16);
    const int n = (N == 128) ? q * 32 + lane : q * 16 + lane;
    if (ok) {
      const float sB_g = a.s_B[g];
      const i64 obase = ((((i64)b * d.c + k) * d.H + h) * P) * N + n;
#pragma unroll
      for (int pp = 0; pp < 32; ++pp) {
        const int p = ch * 32 + pp;
        a.loc[obase + (i64)p * N] = __fmul_rn(i22_to_f32(acc[pp]), __fmul_rn(a.s_xs[h * P + p], sB_g));
        if (a.tap_acc) a.tap_acc[obase + (i64)p * N] = acc[pp];
      }
    }
  }
  tc_fence_before();
  drain_after_timeout(a.status);
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 64);
  }
}

}  // namespace

ssdi8_status_t launch_chunk_state(const Dims& d, const int8_t* xq, const int8_t* Bq,
                                  const float* s_x, const float* s_xs, const float* s_B,
                                  const float* pack, float* loc, int8_t* tap_Xsq,
                                  int32_t* tap_acc, uint32_t* absmax_xs, int32_t* status,
                                  cudaStream_t st) {
  const int TQ = d.Q < 128 ? d.Q : 128;
  const uint64_t T = (uint64_t)d.b * d.L;
  CUtensorMap tm_B, tm_x;
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
  StateArgs a = {s_x, s_xs, s_B, pack, loc, tap_Xsq, tap_acc, absmax_xs, status, d};
  const size_t smem = SMEM_BYTES + 1024;
  SSDI8_CUDA_CHECK(cudaFuncSetAttribute(chunk_state_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid(d.H, d.c, d.b);
  chunk_state_tc<<<grid, kThreads, smem, st>>>(tm_B, tm_x, a);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

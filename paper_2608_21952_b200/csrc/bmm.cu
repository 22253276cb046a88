// ChunkBMM on the group axis (Section 4.2) on tcgen05 tensor cores:
//   acc_cb[i,j] = sum_n Cq[i,n] Bq[j,n]   per (batch, chunk, group), INT32 exact in TMEM, then one
//   INT32 -> INT8 step  CBq = rne(fmul(float(acc_cb), fdiv(fmul(s_C, s_B), s_cb))).
// One CTA per 128-row tile of the chunk; only the columns that touch the causal half are
// computed (row tile it needs columns j < 128 (it + 1)), and within those the 16-column sub-blocks
// after a row's own are stored as zeros.  Both operands are K-major as they sit
// in HBM ([token][N], N contiguous): TMA stages them in the 128-byte (64-byte for N = 64)
// swizzled layout the MMA reads.  The int8 codes leave through a swizzled staging panel and one
// TMA store per 128-column panel.
#include "kernels.h"
#include "sm100.cuh"

namespace ssdi8 {
namespace {

using namespace sm100;

struct BmmArgs {
  const float* s_C; const float* s_B; const float* s_cb;
  int32_t* tap_acc; uint32_t* absmax_acc; int32_t* status;
  Dims d;
  int store;  // 0: calibration pass (no CBq written)
  int late_wait;  // 1: launched right after the fused state kernel, which it does not depend on (see below)
};

constexpr int kThreads = 512;   // 16 warps: warp w reads TMEM lane quarter w % 4 (rows) and every fourth 32-column piece from w / 4
constexpr uint32_t OFF_A = 0;        // [128][N]  Cq rows of the tile
constexpr uint32_t OFF_B = 16384;    // [256][N]  Bq rows 0 .. KJ-1
constexpr uint32_t OFF_O = 49152;    // 2 x [128][128] int8 staging panels
constexpr uint32_t OFF_BAR = 81920;
constexpr uint32_t SMEM_BYTES = OFF_BAR + 64;

__global__ void __launch_bounds__(kThreads)
bmm_tc(const __grid_constant__ CUtensorMap tm_C, const __grid_constant__ CUtensorMap tm_B,
       const __grid_constant__ CUtensorMap tm_o, const BmmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const Dims& d = a.d;
  const int Q = d.Q, N = d.N;
  const int TM = Q < 128 ? Q : 128;
  const int ntile = Q / TM;
  const int it = blockIdx.x % ntile;
  int u = blockIdx.x / ntile;
  const int g = u % d.G;
  const int bk = u / d.G;  // b * c + k
  const int KJ = (it + 1) * TM;  // columns computed by this row tile
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const i64 tok0 = (i64)bk * Q;  // b * L + k * Q
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);  // [0] operands, [1] MMA done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);

  if (tid == 0) {
    mbar_init(&bars[0], 1);
    mbar_init(&bars[1], 1);
    fence_mbar_init();
    tma_prefetch_desc(&tm_C); tma_prefetch_desc(&tm_B); tma_prefetch_desc(&tm_o);
  }
  pdl_launch_dependents();
  if (warp == 1) tmem_alloc(tmem_slot, 256);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // Programmatic dependent launch.  Normally: wait for the predecessor before the first global access.
  // Launched right after the fused state kernel (which waits for ITS predecessor before it lets this
  // kernel be scheduled), the work below runs beside that kernel's last wave, and the wait moves to
  // the end, where it only keeps "this kernel complete" implying "the state kernel complete" for the
  // scan kernel that follows.
  if (!a.late_wait) pdl_wait();

  if (tid == 0) {
    mbar_expect_tx(&bars[0], (uint32_t)(TM * N + KJ * N));
    tma_load_3d(smem + OFF_A, &tm_C, &bars[0], 0, g, (int)(tok0 + it * TM));
    for (int j0 = 0; j0 < KJ; j0 += TM) tma_load_3d(smem + OFF_B + j0 * N, &tm_B, &bars[0], 0, g, (int)(tok0 + j0));
    mbar_wait(&bars[0], 0, a.status);
    tc_fence_after();
    const uint32_t idesc = idesc_s8(128, KJ, 0, 0);  // N = 64, 128 or 256 columns
    for (int s = 0; s < N / 32; ++s)
      mma_s8_ss(tmem, tile_desc(smem_u32(smem + OFF_A) + 32 * s, (uint32_t)N),
                tile_desc(smem_u32(smem + OFF_B) + 32 * s, (uint32_t)N), idesc, s > 0);
    mma_commit(&bars[1]);
  }
  __syncwarp();
  mbar_wait(&bars[1], 0, a.status);
  tc_fence_after();

  // ---- epilogue: thread = row i of the tile, 32 columns at a time; the four warps that share a
  // lane quarter take alternate 32-column pieces
  const float r_cb = a.s_cb ? __fdiv_rn(__fmul_rn(a.s_C[g], a.s_B[g]), a.s_cb[g]) : 0.f;
  const int wq = warp & 3, wc = warp >> 2;
  const int r = wq * 32 + lane;
  const int i = it * TM + r;
  const bool ok = r < TM;
  const uint32_t RBO = (uint32_t)TM;  // row bytes of a staging panel (128, or 64 when Q = 64)
  int amax = 0;
  const i64 obase = (((i64)bk * d.G + g) * Q + i) * Q;
#pragma unroll 1
  for (int j0 = wc * 32; j0 < KJ; j0 += 32 * (kThreads / 128)) {
    int acc[32];
    tmem_ld32(tmem + ((uint32_t)(wq * 32) << 16) + (uint32_t)j0, acc);
    tmem_ld_wait();
    if (ok) {
      uint32_t o[8];
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        uint32_t q4[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int v = acc[w * 4 + e];
          q4[e] = rne_clamp_bits(__fmul_rn(i22_to_f32(v), r_cb));
          if (j0 + w * 4 + e <= i) amax = max(amax, abs(v));
        }
        o[w] = pack4_bits(q4[0], q4[1], q4[2], q4[3]);
      }
      if (a.store) {
        uint8_t* panel = smem + OFF_O + (uint32_t)(j0 / 128) * 16384u;
        const uint32_t c0 = (uint32_t)(j0 % 128) >> 4;  // first 16-byte chunk of this piece in the panel row
        // 16-column sub-blocks that lie wholly above the row's own are written as zeros: the scan
        // kernel builds its masked operand in place over this tile and then has nothing to clear there
        const bool z0 = (j0 >> 4) > (i >> 4), z1 = (j0 >> 4) + 1 > (i >> 4);
        const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
        *reinterpret_cast<uint4*>(panel + swz_off((uint32_t)r, c0, RBO)) = z0 ? zero4 : make_uint4(o[0], o[1], o[2], o[3]);
        *reinterpret_cast<uint4*>(panel + swz_off((uint32_t)r, c0 + 1, RBO)) = z1 ? zero4 : make_uint4(o[4], o[5], o[6], o[7]);
      }
      if (a.tap_acc) {
#pragma unroll
        for (int e = 0; e < 32; ++e) a.tap_acc[obase + j0 + e] = acc[e];
      }
    }
  }
  if (a.absmax_acc) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if (lane == 0) atomicMax(a.absmax_acc + g, (uint32_t)amax);
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && a.store) {
    for (int pn = 0; pn * 128 < KJ; ++pn)
      tma_store_2d(&tm_o, smem + OFF_O + pn * 16384, pn * 128, (int)((((i64)bk * d.G + g) * Q) + it * TM));
    tma_store_commit();
    tma_store_wait_read();
  }
  drain_after_timeout(a.status);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
  // (in the grid's last block only: one waiting block is enough for "this kernel complete" to imply "the state
  // kernel complete", and a wait in every block would keep the blocks of the first wave resident, and the rest
  // of a larger grid unscheduled, until the state kernel has finished)
  if (a.late_wait && blockIdx.x == gridDim.x - 1) pdl_wait();
}

}  // namespace

ssdi8_status_t launch_bmm(const Dims& d, const int8_t* Cq, const int8_t* Bq, const float* s_C,
                          const float* s_B, const float* s_cb, int8_t* CBq, int32_t* tap_acc,
                          uint32_t* absmax_acc, int32_t* status, cudaStream_t st, bool after_state_kernel) {
  const int TM = d.Q < 128 ? d.Q : 128;
  const uint64_t T = (uint64_t)d.b * d.L;
  CUtensorMap tm_C, tm_B, tm_o;
  uint64_t dims[3] = {(uint64_t)d.N, (uint64_t)d.G, T};
  uint64_t str[2] = {(uint64_t)d.N, (uint64_t)d.G * d.N};
  uint32_t box[3] = {(uint32_t)d.N, 1, (uint32_t)TM};
  if (!encode_tensor_map(&tm_C, Cq, 1, 3, dims, str, box, d.N)) return SSDI8_ERR_CUDA;
  if (!encode_tensor_map(&tm_B, Bq, 1, 3, dims, str, box, d.N)) return SSDI8_ERR_CUDA;
  const bool store = s_cb != nullptr && CBq != nullptr;
  {
    // the calibration pass stores nothing; its map points at Cq only so that the encode is valid
    const void* base = store ? (const void*)CBq : (const void*)Cq;
    uint64_t odims[2] = {(uint64_t)d.Q, (uint64_t)d.b * d.c * d.G * d.Q};
    uint64_t ostr[1] = {(uint64_t)d.Q};
    uint32_t obox[2] = {(uint32_t)TM, (uint32_t)TM};
    if (!encode_tensor_map(&tm_o, base, 1, 2, odims, ostr, obox, TM)) return SSDI8_ERR_CUDA;
  }
  BmmArgs a = {s_C, s_B, s_cb, tap_acc, absmax_acc, status, d, store ? 1 : 0, after_state_kernel ? 1 : 0};
  const size_t smem = SMEM_BYTES + 1024;
  SSDI8_CUDA_CHECK(cudaFuncSetAttribute(bmm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const unsigned grid = (unsigned)((i64)d.b * d.c * d.G * (d.Q / TM));
  if (launch_pdl(bmm_tc, dim3(grid), dim3(kThreads), smem, st, tm_C, tm_B, tm_o, a) != cudaSuccess) return SSDI8_ERR_CUDA;
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

}  // namespace ssdi8

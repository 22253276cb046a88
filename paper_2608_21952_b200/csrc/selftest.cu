// Two small kernels beside the layer's own: a dense INT8 tensor-core loop that measures what
// tcgen05.mma.kind::i8 sustains on this device (the denominator of the "fraction of the int8
// tensor-pipe peak" the benchmark reports), and a one-thread kernel that lets a bounded mbarrier
// wait run out on purpose-built, harmless terms so that the time-out path of every kernel
// (status word, normal exit) is exercised by a test.
#include "kernels.h"
#include "sm100.cuh"

namespace ssdi8 {
namespace {

using namespace sm100;

constexpr int kPeakThreads = 128;
constexpr uint32_t PK_OFF_A = 0;        // [128 rows][128 B] int8, 128-byte swizzle: M = 128, K = 128
constexpr uint32_t PK_OFF_B = 16384;    // [256 rows][128 B]: N = 256, K = 128
constexpr uint32_t PK_OFF_BAR = 49152;
constexpr uint32_t PK_SMEM = PK_OFF_BAR + 64;
constexpr int kBatch = 128;             // MMAs between two commits

// Operands stay resident in shared memory (their contents do not matter to the tensor pipe), two
// accumulators of 256 columns alternate so that consecutive batches do not depend on each other,
// one thread issues M 128 x N 256 x K 32 MMAs back to back.  A commit every kBatch MMAs on
// alternating barriers bounds the number of MMAs in flight without draining the pipe.
__global__ void __launch_bounds__(kPeakThreads) int8_mma_peak(int nbatch, int32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + PK_OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
  for (uint32_t o = tid * 16; o < PK_OFF_BAR; o += kPeakThreads * 16)
    *reinterpret_cast<uint4*>(smem + o) = make_uint4(0x01ff0201u, 0xfe0301ffu, 0x0102ff01u, 0xff01fe02u);
  if (tid == 0) {
    mbar_init(&bars[0], 1);
    mbar_init(&bars[1], 1);
    fence_mbar_init();
  }
  if (warp == 1) tmem_alloc(tmem_slot, 512);
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (tid == 0) {
    const uint32_t idesc = idesc_s8(128, 256, 0, 0);
    const uint64_t da0 = tile_desc(smem_u32(smem + PK_OFF_A), 128), db0 = tile_desc(smem_u32(smem + PK_OFF_B), 128);
    for (int bt = 0; bt < nbatch; ++bt) {
      if (bt >= 2) mbar_wait(&bars[bt & 1], ((bt - 2) >> 1) & 1, status);   // batch bt - 2 has left the pipe
      const uint32_t acc = tmem + (uint32_t)(bt & 1) * 256u;
#pragma unroll 4
      for (int m = 0; m < kBatch; ++m) mma_s8_ss(acc, da0 + 2 * (m & 3), db0 + 2 * (m & 3), idesc, m > 0);
      mma_commit(&bars[bt & 1]);
    }
    for (int bt = (nbatch >= 2 ? nbatch - 2 : 0); bt < nbatch; ++bt) mbar_wait(&bars[bt & 1], (bt >> 1) & 1, status);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// One thread initialises a barrier that nothing ever arrives on and waits on it through the
// library's own bounded wait with a cap of 48 polls (each poll is suspended by the hardware for at
// most its 20 us hint, so the kernel ends within about a millisecond).  No copy is in flight, no
// tensor memory is held, nothing can fault: the wait gives up, writes SSDI8_ERR_DEVICE_TIMEOUT to the
// status word and the kernel returns normally.
__global__ void bounded_wait_expires(int32_t* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_mbar_init();
    mbar_wait_slow<48>(&bar, 0, status, 0u);
  }
}

}  // namespace

ssdi8_status_t launch_int8_mma_peak(int nbatch, int32_t* status, int* ctas, cudaStream_t st) {
  int dev = 0, sms = 0;
  SSDI8_CUDA_CHECK(cudaGetDevice(&dev));
  SSDI8_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const size_t smem = PK_SMEM + 1024;
  SSDI8_CUDA_CHECK(cudaFuncSetAttribute(int8_mma_peak, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  int8_mma_peak<<<sms, kPeakThreads, smem, st>>>(nbatch, status);
  SSDI8_LAUNCH_CHECK();
  *ctas = sms;
  return SSDI8_OK;
}

ssdi8_status_t launch_bounded_wait_expires(int32_t* status, cudaStream_t st) {
  bounded_wait_expires<<<1, 32, 0, st>>>(status);
  SSDI8_LAUNCH_CHECK();
  return SSDI8_OK;
}

int int8_mma_peak_batch() { return kBatch; }

}  // namespace ssdi8

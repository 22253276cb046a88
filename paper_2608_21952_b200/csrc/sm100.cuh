// Blackwell (sm_100a) primitives used by the tensor-core kernels: mbarriers with bounded
// waits, TMA tile copies, tensor-memory allocation, tcgen05 MMA issue/commit and
// tensor-memory loads, and the shared-memory / instruction descriptors for 8-bit operands.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace ssdi8 {
namespace sm100 {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// ------------------------------------------------------------------ mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One attempt: the thread is suspended by the hardware until the phase completes or the
// suspend-time hint (about 20 us here) runs out, so a waiting warp does not burn issue slots.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(20000u)
      : "memory");
  return ok != 0;
}
// One look at the barrier without suspending: has the phase of that parity completed?
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Every try_wait blocks for up to its suspend-time hint, so the cap is of the
// order of a second.  On expiry the caller's status word is set and the wait returns; once
// the word is set, every later wait of the grid gives up after a few polls, so the kernel runs
// to its normal end (tensor memory is freed) quickly, with undefined results.
// The polling loop is one out-of-line function: a call site is the first attempt and a branch, so
// the many waits of a warp-specialised kernel do not bloat its instruction footprint.
constexpr uint32_t kWaitCap = 1u << 17;
// (CAP is a template parameter only so that the library's self-test can run this very loop with a
// cap of a few dozen polls on a barrier nobody arrives on; every kernel of the layer uses kWaitCap.)
template <uint32_t CAP = kWaitCap>
static __device__ __noinline__ void mbar_wait_slow(uint64_t* bar, uint32_t parity, int32_t* status,
                                                   uint32_t sleep_ns) {
  for (uint32_t it = 0; it < CAP; ++it) {
    if (mbar_try_wait(bar, parity)) return;
    if (sleep_ns) __nanosleep(sleep_ns);
    if ((it & 255u) == 255u && status && *reinterpret_cast<volatile int32_t*>(status) != 0) return;
  }
  if (status) atomicExch(status, (int32_t)SSDI8_ERR_DEVICE_TIMEOUT);
}
__device__ __forceinline__ void mbar_wait(uint64_t* bar, uint32_t parity, int32_t* status) {
  if (!mbar_try_wait(bar, parity)) mbar_wait_slow(bar, parity, status, 0u);
}

// The same bounded wait for warps whose wait is long and off the critical path (producers waiting
// for a free slot, epilogue warps waiting for an accumulator): a failed poll is followed by a short
// sleep, so the polling loop leaves the issue slots to the warps that compute.
__device__ __forceinline__ void mbar_wait_relaxed(uint64_t* bar, uint32_t parity, int32_t* status) {
  if (!mbar_try_wait(bar, parity)) mbar_wait_slow(bar, parity, status, 256u);
}

// named barrier among `nthreads` threads (whole warps) of the CTA; id 0 is __syncthreads
__device__ __forceinline__ void named_bar_sync(uint32_t id, uint32_t nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// At the end of a kernel whose waits are bounded: if some wait of the grid gave up (the status word is
// set), the handshakes of this CTA may be broken and copies into its shared memory may still be in
// flight; give them a bounded time to land before the CTA retires and its shared memory is handed on.
__device__ __forceinline__ void drain_after_timeout(const int32_t* status) {
  if (status && *reinterpret_cast<const volatile int32_t*>(status) != 0)
    for (int i = 0; i < 50; ++i) __nanosleep(1000);
}

// Inline forms of both waits, for kernels with few wait sites and no registers to spare around a call.
template <uint32_t SLEEP_NS>
__device__ __forceinline__ void mbar_wait_inline(uint64_t* bar, uint32_t parity, int32_t* status) {
  for (uint32_t it = 0; it < kWaitCap; ++it) {
    if (mbar_try_wait(bar, parity)) return;
    if (SLEEP_NS) __nanosleep(SLEEP_NS);
    if ((it & 255u) == 255u && status && *reinterpret_cast<volatile int32_t*>(status) != 0) return;
  }
  if (status) atomicExch(status, (int32_t)SSDI8_ERR_DEVICE_TIMEOUT);
}

// ------------------------------------------------------------------ proxies and fences
__device__ __forceinline__ void fence_async_smem() {  // generic-proxy smem writes -> async proxy
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// ------------------------------------------------------------------ TMA (no multicast anywhere)
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, uint64_t* bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* tm, uint64_t* bar, int x, int y,
                                            int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}
// untiled bulk copy global -> shared (both 16-byte aligned, size a multiple of 16)
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tm, const void* src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(tm), "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z)
               : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, const void* src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(tm), "r"(smem_u32(src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
// all but the most recent bulk store of this thread have finished reading shared memory
__device__ __forceinline__ void tma_store_wait_read1() {
  asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

// ------------------------------------------------------------------ tensor memory
// One full warp allocates / frees; `ncols` is a power of two in [32, 512].
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)),
               "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp receives lane (base + t).
// The lane field of taddr must be the first lane of the warp's quarter (32 * (warp % 4)).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, int (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, int (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, int (&v)[8]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 32 lanes x 8 consecutive 32-bit columns, registers -> tensor memory (thread t writes lane base + t)
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const int (&v)[8]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ------------------------------------------------------------------ descriptors
// Shared-memory matrix descriptor (64 bit): start address, leading and stride byte offsets
// in 16-byte units, descriptor version 1, swizzle mode.
enum : uint32_t { SWZ_NONE = 0, SWZ_128B = 2, SWZ_64B = 4, SWZ_32B = 6 };

__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                              uint32_t swizzle) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)swizzle << 61);
}

// Operand tile whose rows are `row_bytes` (64 or 128) long and swizzled at that width: rows are
// the M/N index for a K-major operand and the K index for an MN-major operand.  Groups of 8
// rows are `8 * row_bytes` apart (the stride byte offset) in both cases.
__device__ __forceinline__ uint64_t tile_desc(uint32_t saddr, uint32_t row_bytes) {
  return smem_desc(saddr, 16, 8 * row_bytes, row_bytes == 128 ? SWZ_128B : SWZ_64B);
}

// Instruction descriptor for kind::i8: signed 8-bit A and B, 32-bit integer accumulator.
__host__ __device__ constexpr uint32_t idesc_s8(int M, int N, int a_mn_major, int b_mn_major) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) |
         ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]; issued by one thread.
__device__ __forceinline__ void mma_s8_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// All MMAs issued so far by this thread arrive on `bar` when they have completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// byte offset of 16-byte chunk `c` of row `r` inside a swizzled tile with rows of `row_bytes`
__device__ __forceinline__ uint32_t swz_off(uint32_t r, uint32_t c, uint32_t row_bytes) {
  return row_bytes == 128 ? r * 128u + ((c ^ (r & 7u)) << 4) : r * 64u + ((c ^ ((r >> 1) & 3u)) << 4);
}

}  // namespace sm100

// ------------------------------------------------------------------ host: tensor maps
// Encodes a tiled tensor map over 8-bit or 32-bit elements (dims innermost first).  Returns
// false if the driver entry point is unavailable or the encode fails.
bool encode_tensor_map(CUtensorMap* out, const void* base, int elem_bytes, int rank, const uint64_t* dims,
                       const uint64_t* strides_bytes /* rank-1 entries */, const uint32_t* box,
                       int swizzle_bytes /* 0, 64, 128 */);

}  // namespace ssdi8

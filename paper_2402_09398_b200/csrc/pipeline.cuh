// Shared-memory pipelines fed by bulk asynchronous copies (TMA, 1-D form):
// mbarrier and cp.async.bulk wrappers.  Every wait is bounded: after
// kSpinLimit polls the waiter gives up, and the caller sets the device status
// word and leaves, so a mistake can never hang the GPU.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace less {

constexpr uint32_t kSpinLimit = 1u << 26;   // ~ a second of polling at most

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

// makes freshly initialised barriers visible to the async proxy (bulk copies, MMA commits)
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// One arrival for a whole warp: every lane has finished (and fenced) its own accesses, the
// warp converges, lane 0 arrives.  Barriers counted in warps avoid hundreds of serialised
// arrivals on one shared-memory word.
__device__ __forceinline__ void mbar_arrive_warp(uint64_t* bar) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait for the phase with the given parity to complete.  false = gave up after `limit` polls.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t limit = kSpinLimit) {
  for (uint32_t i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

// The wait every pipeline role uses.  Fast path: the phase is already complete.  Otherwise the
// waiter leaves at once if its CTA has given up; a wait that runs out makes the CTA give up and
// records where in the device status word (first writer wins), so that nothing can hang.
__device__ __forceinline__ void wait_or_give_up(uint64_t* bar, uint32_t parity, volatile int* abort, int32_t* status,
                                                int where, uint32_t limit = kSpinLimit) {
  if (mbar_try_wait(bar, parity)) return;
  if (*abort) return;
  if (!mbar_wait(bar, parity, limit)) {
    *abort = 1;
    if (atomicCAS(status, 0, 1 /* timeout */) == 0) status[1] = where;
  }
}

// Error path only: a CTA that gave up on a wait lets its bulk copies and MMAs in flight land
// (a bounded pause, ~0.25 ms) before it releases shared and tensor memory.
__device__ __forceinline__ void drain_after_abort(volatile int* abort) {
  if (*abort)
    for (int i = 0; i < 64; ++i) __nanosleep(4000);
}

// 1-D bulk copy global -> shared; completes `bytes` on the barrier.
// dst, src 16-byte aligned; bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes,
                                         uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst_smem)),
      "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// orders generic-proxy accesses to shared memory before later async-proxy accesses
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

}  // namespace less

// mbarrier and bulk-copy (TMA, untiled) primitives for shared-memory pipelines on sm_100a.
//
// Every wait is bounded: after `limit` failed polls (kSpinLimit unless the context was given another value through
// ckv_debug_set) the wait gives up and returns false, and the caller records CKV_DEV_TIMEOUT and drains its
// outstanding copies before leaving.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ckv_pipe {

constexpr uint32_t kSpinLimit = 1u << 22;   // polls; each poll may itself block for a short hardware-defined time

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
// Makes the initialised barriers visible to the async (bulk-copy) proxy.
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
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
// Bounded wait for the phase with the given parity to complete.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, uint32_t limit = kSpinLimit) {
  for (uint32_t i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// Global -> shared bulk copy; completion is signalled on `bar` as `bytes` transaction bytes.
// dst, src and bytes must be multiples of 16.
__device__ __forceinline__ void bulk_g2s(void *dst_smem, const void *src_gmem, uint32_t bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// bulk_g2s with its arguments checked first: a copy that is misaligned, empty or would leave the window
// [smem_lo, smem_hi) is not issued and the function returns false (the caller records the fault; the
// barrier then never completes and the bounded waits on it run out).
__device__ __forceinline__ bool bulk_g2s_checked(void *dst_smem, const void *src_gmem, uint32_t bytes, uint64_t *bar,
                                                 uint32_t smem_lo, uint32_t smem_hi) {
  const uint32_t d = smem_u32(dst_smem);
  const bool ok = bytes != 0 && (bytes & 15u) == 0 && (d & 15u) == 0 && ((unsigned long long)src_gmem & 15ull) == 0 &&
                  d >= smem_lo && d + bytes <= smem_hi;
  if (ok) bulk_g2s(dst_smem, src_gmem, bytes, bar);
  return ok;
}
// Orders this thread's earlier generic-proxy accesses to shared memory before later async-proxy
// (bulk copy) accesses to it.
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// Barrier among a subset of the CTA's warps (id 1..15; count a multiple of 32).
__device__ __forceinline__ void named_barrier(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

}  // namespace ckv_pipe

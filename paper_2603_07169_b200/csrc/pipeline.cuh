// mbarrier + bulk-copy (TMA, 1-D) helpers for the shared-memory staging pipelines.
// Every wait is bounded: after `limit` polls (option "spin_limit", default kSpinLimit) the caller records an error and leaves.
#pragma once
#include "common.cuh"

namespace b200sp {

constexpr int kSpinLimit = 1 << 20;  // polls of try_wait (each may block for a hardware-defined time slice)

__device__ __forceinline__ unsigned smem_addr(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Returns false if the barrier did not flip within `limit` polls.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity, int limit) {
  for (int spin = 0; spin < limit; ++spin)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// Orders this thread's earlier generic-proxy accesses to shared memory (and, through a preceding CTA
// barrier, those of the other threads) before the async-proxy writes of bulk copies issued after it.
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Global -> shared bulk copy; src and dst 16-byte aligned, bytes a positive multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

}  // namespace b200sp

// One-instruction wrappers around the asynchronous-copy machinery of sm_100a used by the staged row
// kernels: mbarriers in shared memory, 1-D bulk copies global <-> shared (no multicast anywhere),
// the global nanosecond timer that bounds every wait.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace codistill {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
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
// global -> shared bulk copy (no multicast); dst, src and bytes are multiples of 16
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// shared -> global bulk copy; dst, src and bytes are multiples of 16.  Completion is tracked by the
// issuing thread's bulk async-group.
__device__ __forceinline__ void bulk_s2g(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all_groups() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// orders this thread's earlier generic-proxy writes to shared memory before later bulk (async-proxy) reads of them
__device__ __forceinline__ void fence_proxy_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait for a phase of an mbarrier.  Polls until the phase completes, or the CTA-wide abort flag is
// up (only when heed_abort), or `limit_ns` nanoseconds of polling have gone by; in the last case it raises the
// abort flag and ORs `timeout_bit` into *status.  Returns true when the phase completed.  With back_off the
// thread sleeps between polls (for warps that have slack and should not take issue slots from others).
// Kept out of line: callers try the barrier once inline and come here only when they really have to wait.
static __device__ __noinline__ bool mbar_wait_limited(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status,
                                               int timeout_bit, unsigned long long limit_ns, bool heed_abort, bool back_off) {
  uint32_t polls = 0;
  unsigned long long t0 = 0;
  while (!mbar_try_wait(bar, parity)) {
    if (back_off) __nanosleep(128);
    if ((++polls & 0x3FFu) == 0 || (back_off && (polls & 0x3Fu) == 0)) {
      if (heed_abort && *abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > limit_ns) {
        *abort_flag = 1;
        atomicOr(status, timeout_bit);
        return false;
      }
    }
  }
  return true;
}

}  // namespace codistill

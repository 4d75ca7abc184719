// mbarrier and timer helpers shared by the kernels that stage data with TMA (sm_100a).
// Every wait is bounded: it gives up after kWaitLimitNs, or as soon as another thread has
// recorded a failure in the status word, and reports that to the caller.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace fly {

// Far above any legitimate wait (a tile takes ~70 us).  %globaltimer also runs while the context is
// preempted or time-sliced with another process, so on a shared GPU a wait can in principle run out
// without a fault in the kernel: the limit is generous for that reason, and a run-out is reported,
// never trapped on.
constexpr unsigned long long kWaitLimitNs = 200ull * 1000 * 1000;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Waits for the phase of `bar` with the given parity to complete.  Gives up when
// the limit passes or when another role has already reported a failure.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* status, int code,
                                          unsigned long long limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63) == 0) {
      if (*(volatile int*)status != 0) return false;
      if (global_ns() - t0 > limit_ns) {
        atomicCAS(status, 0, code);
        return false;
      }
    }
  }
  return true;
}

// The same wait without a status word: for the give-up path, where the failure is already recorded.
__device__ __forceinline__ bool mbar_wait_quiet(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63) == 0 && global_ns() - t0 > limit_ns) return false;
  }
  return true;
}

}  // namespace fly

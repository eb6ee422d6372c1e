// Thin wrappers over the PTX used by the asynchronous-copy pipelines: mbarrier, bulk copy
// (TMA engine, 1-D form) and bounded waits.
#pragma once

#include "common.cuh"

namespace phyai {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}

struct WaitCtx {
  int* status;
  volatile int* abort_flag;  // shared memory, CTA-wide
  uint32_t limit;
};
// Bounded wait.  Returns false (and records ST_TIMEOUT) when the limit expires or the CTA has
// already given up; callers then skip their side effects but keep walking their loops.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& c) {
  if (mbar_test(bar, parity)) return true;   // fast path: already complete
  if (*c.abort_flag) return false;
  for (uint32_t it = 0; it < c.limit; ++it) {
    if (mbar_test(bar, parity)) return true;
    // Back off only when the wait is clearly not a pipeline wait of a few microseconds: a warp that sleeps wakes up
    // late (measured: 0.75 us from an arrival to the waiting warp's next instruction with a 32 ns sleep in the loop,
    // which every hand-over inside the batch-1 kernels paid).
    if (it > 8192) __nanosleep(64);
  }
  *c.abort_flag = 1;
  atomicExch(c.status, ST_TIMEOUT);
  return false;
}

// Wait on a barrier behind which asynchronous copies into this CTA's shared memory (or tensor-core reads of it) are
// outstanding.  The caller's limit decides when the call is given up (status word raised, side effects suppressed);
// the shared memory, however, may only be released once those copies have landed, so the wait then continues under a
// generous bound of its own.  Returns 1 = completed in time, 0 = given up but the barrier did complete, -1 = not even
// within the drain bound.  Kernels keep their copy / MMA / commit protocol going after a 0, so every barrier of the
// pipeline still completes; only global stores are skipped.
constexpr uint32_t DRAIN_LIMIT = 1u << 22;
__device__ __forceinline__ int mbar_wait_drain(uint32_t bar, uint32_t parity, const WaitCtx& c) {
  if (mbar_wait(bar, parity, c)) return 1;
  for (uint32_t it = 0; it < DRAIN_LIMIT; ++it) {
    if (mbar_test(bar, parity)) return 0;
    __nanosleep(64);
  }
  return -1;
}

__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}


}  // namespace phyai

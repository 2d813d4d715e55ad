// Asynchronous bulk copies from global to shared memory (cp.async.bulk, the copy engine that also serves tensor
// maps) and the mbarrier objects that report their completion: thin wrappers over the PTX, CTA-local use only.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace cpe {

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void ac_mbar_init(uint32_t mbar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count) : "memory");
}
// Makes freshly initialised barriers visible to the asynchronous proxy; follow with a CTA barrier.
__device__ __forceinline__ void ac_fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

__device__ __forceinline__ void ac_mbar_arrive(uint32_t mbar) {
  asm volatile("{\n.reg .b64 st;\nmbarrier.arrive.shared::cta.b64 st, [%0];\n}\n" ::"r"(mbar) : "memory");
}
// One arrival that also announces `bytes` of asynchronous copies whose completion the phase has to wait for.
__device__ __forceinline__ void ac_mbar_arrive_expect_tx(uint32_t mbar, uint32_t bytes) {
  asm volatile("{\n.reg .b64 st;\nmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}\n" ::"r"(mbar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool ac_mbar_try_wait(uint32_t mbar, uint32_t parity) {
  uint32_t done;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(done) : "r"(mbar), "r"(parity) : "memory");
  return done != 0;
}
// Bounded wait for the phase of the given parity; gives up early once the CTA's abort flag is up.  False: gave up.
constexpr int kAcWaitLimit = 1 << 22;
__device__ __forceinline__ bool ac_mbar_wait(uint32_t mbar, uint32_t parity, const volatile int* abort_flag,
                                             int limit = kAcWaitLimit) {
  for (int it = 0; it < limit; ++it) {
    if (ac_mbar_try_wait(mbar, parity)) return true;
    if ((it & 15) == 15 && *abort_flag) return false;
  }
  return false;
}

// `bytes` (a multiple of 16) from global `src` to this CTA's shared memory at `dst` (both 16-byte aligned); the
// completion is counted on `mbar`.
__device__ __forceinline__ void ac_bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t mbar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(mbar)
               : "memory");
}

}  // namespace cpe

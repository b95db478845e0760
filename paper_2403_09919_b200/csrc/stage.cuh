// Row segments staged through shared memory with bulk asynchronous copies (cp.async.bulk + mbarrier).
//
// The row-wise kernels of a launch with many rows are bound by the bytes an SM has outstanding.  With register
// loads that number is (resident threads) x (loads each thread can hold), and the bookkeeping of the deferred
// projection reduction leaves few registers for it.  A ring of shared-memory stages filled by one elected thread
// decouples the two: a CTA has STAGES x (segment bytes) in flight whatever its threads are doing.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace rd {

__device__ __forceinline__ uint32_t stage_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void stage_bar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void stage_bar_init_fence() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void stage_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Contiguous copy global -> shared; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void stage_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
               "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ bool stage_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait (one second): on expiry raises `err_bit` in the status word and returns false; the caller carries on
// with whatever the stage holds (the step's results are then void, which the status word says) and leaves normally.
__device__ __forceinline__ bool stage_wait(uint32_t bar, uint32_t parity, int32_t* status, int err_bit) {
  if (stage_try_wait(bar, parity)) return true;
  unsigned long long t0;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
  for (uint32_t it = 1;; ++it) {
    if (stage_try_wait(bar, parity)) return true;
    if ((it & 255u) == 0u) {
      unsigned long long t1;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
      if (t1 - t0 > 1000000000ull) {
        atomicOr(status, err_bit);
        return false;
      }
    }
  }
}

}  // namespace rd

// Counter hand-off between consecutive launches of the decode step.
//
// The step is a fixed chain of launches in one stream, each consuming what the one before it wrote.
// Programmatic dependent launch already lets launch q+1 become resident while launch q runs, but its
// `griddepcontrol.wait` returns only after launch q has completely drained and flushed, which costs a
// few microseconds per boundary -- as much as the short kernels' own work.  A chained launch instead
// waits on a counter in device memory: every CTA of launch q adds one to its counter after its last
// store (release), launch q+1 polls until the counter reaches the number of CTAs of launch q (acquire).
// Because launch q+1 cannot start before every CTA of launch q is resident (that is what the
// programmatic launch guarantees) and a CTA only ever waits on EARLIER launches, the polls cannot
// deadlock; they are bounded all the same and raise DEV_ERR_TIMEOUT.
//
// Ordering is transitive: a CTA of launch q signals only after it has itself seen launch q-1 complete,
// so a launch that observes its predecessor's counter may also rely on everything before it.
// A launch with wait_ptr == nullptr falls back to the grid dependency (used after un-chained launches).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "pdl.cuh"

namespace rd {

constexpr int CHAIN_SLOTS = 16;  // counters in rotation; a counter is reused 16 launches later, and only grows

struct ChainSync {
  const unsigned int* wait_ptr;   // counter of the preceding chained launch, or nullptr: wait on the grid dependency
  unsigned int wait_target;       // value it reaches when every CTA of that launch has signalled
  unsigned int* signal_ptr;       // counter this launch's CTAs add to, or nullptr
  int32_t* status;                // device status word (timeouts)
  unsigned long long* trace;      // 8 timestamps of this launch when tracing (short kernels only) or nullptr
};

// Host-side bookkeeping: hands out (wait, signal) pairs in launch order.
struct Chain {
  unsigned int* ctr = nullptr;    // CHAIN_SLOTS device counters, zeroed once at creation
  int32_t* status = nullptr;
  unsigned int cum[CHAIN_SLOTS] = {};
  int next = 0;
  const unsigned int* prev_ptr = nullptr;
  unsigned int prev_target = 0;
  bool enabled = false;
  // tracing: the short kernels take their timestamp slot here (the projections and attention get theirs from the caller)
  unsigned long long* trace_base = nullptr;
  int* trace_next = nullptr;
  int trace_cap = 0;
  // The next chained launch has n_ctas CTAs, each signalling exactly once.
  ChainSync link(unsigned int n_ctas, bool want_trace = false) {
    ChainSync cs{nullptr, 0u, nullptr, status, nullptr};
    if (want_trace && trace_next && *trace_next >= 0 && *trace_next < trace_cap) cs.trace = trace_base + (size_t)8 * (*trace_next)++;
    if (!enabled || !ctr) return cs;
    cs.wait_ptr = prev_ptr;
    cs.wait_target = prev_target;
    const int s = next;
    next = (next + 1) % CHAIN_SLOTS;
    cum[s] += n_ctas;
    cs.signal_ptr = ctr + s;
    prev_ptr = ctr + s;
    prev_target = cum[s];
    return cs;
  }
  // An un-chained launch follows: whatever comes after it must wait on the grid dependency again.
  void cut() { prev_ptr = nullptr; }
  // Counters and targets back to zero (enqueued on `st`; nothing of the chain may be in flight on another stream).
  // Needed when a launch that link() had already counted never ran, or a wait gave up: the device counters would
  // stay behind their host-side targets for good.
  cudaError_t reset(cudaStream_t st) {
    for (int i = 0; i < CHAIN_SLOTS; ++i) cum[i] = 0;
    next = 0;
    cut();
    return ctr ? cudaMemsetAsync(ctr, 0, CHAIN_SLOTS * sizeof(unsigned int), st) : cudaSuccess;
  }
};

#ifdef __CUDACC__
constexpr unsigned long long CHAIN_WAIT_LIMIT_NS = 1000000000ull;
constexpr int CHAIN_ERR_TIMEOUT = 1 << 2;  // == DEV_ERR_TIMEOUT

__device__ __forceinline__ unsigned int chain_load_acquire(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// One thread: wait until the predecessor has signalled completely (or fall back to the grid dependency).
// Bounded; gives up at once when an earlier wait of the step already timed out.
__device__ __forceinline__ void chain_wait_thread(const ChainSync& cs) {
  if (!cs.wait_ptr) { pdl_wait(); return; }
  if ((int)(chain_load_acquire(cs.wait_ptr) - cs.wait_target) >= 0) return;
  unsigned long long t0;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
  for (unsigned int it = 1;; ++it) {
    if ((int)(chain_load_acquire(cs.wait_ptr) - cs.wait_target) >= 0) return;
    __nanosleep(40);
    if ((it & 255u) == 0u) {
      if (*(volatile int32_t*)cs.status & CHAIN_ERR_TIMEOUT) return;
      unsigned long long t1;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
      if (t1 - t0 > CHAIN_WAIT_LIMIT_NS) { atomicOr(cs.status, CHAIN_ERR_TIMEOUT); return; }
    }
  }
}

// The thread that waited is about to hand the predecessor's data to the TMA unit (asynchronous proxy).
__device__ __forceinline__ void chain_fence_async_reads() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

__device__ __forceinline__ unsigned long long chain_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Whole CTA, first thing in the kernel: let the dependents start.  Between chain_begin and chain_wait_cta a
// kernel may load what no launch of the step writes (weights).
__device__ __forceinline__ void chain_begin(const ChainSync& cs) {
  pdl_launch_dependents();
  const bool t0 = threadIdx.x == 0 && threadIdx.y == 0 && threadIdx.z == 0;
  if (cs.trace && t0) { const unsigned long long t = chain_now(); atomicMin(cs.trace + 0, t); atomicMax(cs.trace + 7, t); }
}
// Whole CTA: wait for the predecessor.
__device__ __forceinline__ void chain_wait_cta(const ChainSync& cs) {
  const bool t0 = threadIdx.x == 0 && threadIdx.y == 0 && threadIdx.z == 0;
  if (!cs.wait_ptr) {
    pdl_wait();
  } else {
    if (t0) chain_wait_thread(cs);
    __syncthreads();
  }
  if (cs.trace && t0) { const unsigned long long t = chain_now(); atomicMin(cs.trace + 1, t); atomicMax(cs.trace + 2, t); }
}
__device__ __forceinline__ void chain_enter(const ChainSync& cs) {
  chain_begin(cs);
  chain_wait_cta(cs);
}

// Whole CTA, exactly once, after its last store (every thread of the CTA must reach this call).
__device__ __forceinline__ void chain_exit(const ChainSync& cs) {
  if (!cs.signal_ptr && !cs.trace) return;
  __syncthreads();
  const bool t0 = threadIdx.x == 0 && threadIdx.y == 0 && threadIdx.z == 0;
  if (cs.trace && t0) { const unsigned long long t = chain_now(); atomicMin(cs.trace + 5, t); atomicMax(cs.trace + 6, t); }
  if (cs.signal_ptr && t0) {
    // release: the CTA's stores (ordered before this thread by the barrier above) become visible before the
    // increment; a consumer that hands the data to the TMA unit adds its own proxy fence after its acquire
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(cs.signal_ptr) : "memory");
  }
}
#endif

}  // namespace rd

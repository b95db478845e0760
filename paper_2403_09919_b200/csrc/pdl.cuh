// Programmatic dependent launch: every kernel of the library is launched with programmatic stream
// serialization, lets its dependents start as early as possible and waits for its predecessors
// before it touches anything they produce.  A kernel may do work that depends on nothing produced
// inside the step (the projection prefetches weights) between the two calls.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <unordered_set>
#include <utility>

namespace rd {

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// For kernels with no independent prologue.
__device__ __forceinline__ void pdl_enter() {
  pdl_launch_dependents();
  pdl_wait();
}

// Every kernel of the library asks for the same split of the SM's L1/shared-memory array (all of it as
// shared memory).  An SM can only change that split while it is empty, so a projection CTA (about 150 KB of
// shared memory) could otherwise not join an SM that still runs a short kernel's CTA configured for a large
// L1: it would have to wait for the SM to drain, and the weight stream it is meant to start early would
// start late.
inline void prefer_max_shared(const void* kernel) {
  static std::mutex mu;
  static std::unordered_set<unsigned long long> done;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return;
  const unsigned long long key = (unsigned long long)(uintptr_t)kernel * 64ull + (unsigned long long)dev;
  std::lock_guard<std::mutex> lock(mu);
  if (done.count(key)) return;
  done.insert(key);
  cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  prefer_max_shared(reinterpret_cast<const void*>(kernel));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(std::forward<Args>(args))...);
}

// The same launch without the programmatic attribute: the kernel starts only when everything before it in
// the stream has completed.  Used for the first launch of a chain, so that every later launch of the chain
// may read, even before its own wait, what the kernels ahead of the chain wrote (row tables, rotary table,
// masks, older cache entries).
template <typename... KArgs, typename... Args>
cudaError_t launch_ordered(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  prefer_max_shared(reinterpret_cast<const void*>(kernel));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = nullptr;
  cfg.numAttrs = 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(std::forward<Args>(args))...);
}

}  // namespace rd

// The fused epilogue every projection kernel applies to one output element.
#pragma once
#include "rd_internal.cuh"

namespace rd {

template <typename T>
__device__ __forceinline__ void apply_epilogue(const Epilogue& ep, int m, int n, float v) {
  if (ep.addend) v += ep.addend[(size_t)m * ep.ld_addend + n];
  if (ep.bias) v += to_f<T>(reinterpret_cast<const T*>(ep.bias)[n]);
  if (ep.silu) v = silu_f(v);
  if (ep.resid) v += ep.resid[(size_t)m * ep.ld_resid + n];
  if (ep.out_f32) ep.out_f32[(size_t)m * ep.ld_out_f32 + n] = v;
  if (ep.out_t) reinterpret_cast<T*>(ep.out_t)[(size_t)m * ep.ld_out_t + n] = from_f<T>(v);
}

}  // namespace rd

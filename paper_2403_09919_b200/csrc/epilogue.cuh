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

// The same epilogue for 16 consecutive rows m0 .. m0+15 of one output column n (rows >= m_end are
// skipped).  All loads are issued before the first store, so they overlap instead of forming a
// chain of L2 round trips (the residual is updated in place, which would otherwise order them).
template <typename T>
__device__ __forceinline__ void apply_epilogue16(const Epilogue& ep, int m0, int m_end, int n, const float (&acc)[16]) {
  float v[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) v[j] = acc[j];
  if (ep.addend) {
    float t[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) t[j] = (m0 + j < m_end) ? ep.addend[(size_t)(m0 + j) * ep.ld_addend + n] : 0.f;
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] += t[j];
  }
  if (ep.bias) {
    const float b = to_f<T>(reinterpret_cast<const T*>(ep.bias)[n]);
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] += b;
  }
  if (ep.silu) {
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = silu_f(v[j]);
  }
  if (ep.resid) {
    float t[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) t[j] = (m0 + j < m_end) ? ep.resid[(size_t)(m0 + j) * ep.ld_resid + n] : 0.f;
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] += t[j];
  }
  if (ep.out_f32) {
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (m0 + j < m_end) ep.out_f32[(size_t)(m0 + j) * ep.ld_out_f32 + n] = v[j];
  }
  if (ep.out_t) {
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (m0 + j < m_end) reinterpret_cast<T*>(ep.out_t)[(size_t)(m0 + j) * ep.ld_out_t + n] = from_f<T>(v[j]);
  }
}

}  // namespace rd

// CUDA-core projection Y[m][n] = sum_k A[m][k] W[n][k] (fp32 result; the consumer applies the epilogue).
//
// Used for the fp32 configuration (no tensor-core path for fp32 operands is wanted there: the
// point of that configuration is tight parity) and for very small M (the autoregressive
// comparator, M = batch), where the projection is a matrix-vector product bound by the weight
// stream: one warp owns one weight row, reads it once with 128-bit loads and keeps MT running
// sums, so the weight is read exactly once per MT rows.
#include "rd_internal.cuh"
#include "pdl.cuh"
#include "gemm_out.cuh"

namespace rd {

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  __device__ static __forceinline__ void load(const float* p, float (&v)[4]) {
    const float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  __device__ static __forceinline__ void load_stream(const float* p, float (&v)[4]) {
    const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static __forceinline__ void unpack(const uint4& t, float (&v)[8]) {
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8]) {
    unpack(*reinterpret_cast<const uint4*>(p), v);
  }
  __device__ static __forceinline__ void load_stream(const __nv_bfloat16* p, float (&v)[8]) {
    unpack(__ldcs(reinterpret_cast<const uint4*>(p)), v);
  }
};

// grid (ceil(N / 8), ceil(m_max / MT)), block 256 = 8 warps, one weight row per warp.
template <typename T, int MT>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T* __restrict__ A, int lda, const T* __restrict__ W, int N,
                                                        int K, const int32_t* __restrict__ m_total, float* __restrict__ raw,
                                                        int ld_raw) {
  pdl_enter();
  constexpr int VN = Vec<T>::N;
  const int M = *m_total;
  const int m0 = blockIdx.y * MT;
  if (m0 >= M) return;
  const int lane = threadIdx.x & 31;
  const int n = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (n >= N) return;
  const int rows = min(MT, M - m0);
  float acc[MT];
#pragma unroll
  for (int r = 0; r < MT; ++r) acc[r] = 0.f;
  const T* wrow = W + (size_t)n * K;
  for (int k = lane * VN; k < K; k += 32 * VN) {
    float w[VN];
    Vec<T>::load_stream(wrow + k, w);
#pragma unroll
    for (int r = 0; r < MT; ++r) {
      if (r < rows) {
        float a[VN];
        Vec<T>::load(A + (size_t)(m0 + r) * lda + k, a);
#pragma unroll
        for (int i = 0; i < VN; ++i) acc[r] = fmaf(a[i], w[i], acc[r]);
      }
    }
  }
#pragma unroll
  for (int r = 0; r < MT; ++r) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], o);
  }
#pragma unroll
  for (int r = 0; r < MT; ++r)
    if (lane == r && r < rows) raw[(size_t)(m0 + r) * ld_raw + n] = acc[r];
}

cudaError_t launch_gemm_simt(int dtype, const void* A, int lda, const void* W, int N, int K, const int32_t* m_total,
                             int m_max, float* raw, int ld_raw, GemmOut* out_desc, cudaStream_t st) {
  if (out_desc) {
    out_desc->raw = raw; out_desc->partial = nullptr; out_desc->ld = ld_raw; out_desc->nkb = 1; out_desc->n_tiles = 1;
    out_desc->mt = 1; out_desc->grid = 1; out_desc->m_tiles_max = 1; out_desc->all_work = 1; out_desc->pair = 0; out_desc->small32 = 0;
  }
  if (m_max <= 0) return cudaSuccess;
  if (m_max <= 2) {
    dim3 grid((N + 7) / 8, (m_max + 1) / 2);
    if (dtype == RD_DTYPE_FP32)
      launch_pdl(gemm_simt_kernel<float, 2>, grid, 256, 0, st, (const float*)A, lda, (const float*)W, N, K, m_total, raw, ld_raw);
    else
      launch_pdl(gemm_simt_kernel<__nv_bfloat16, 2>, grid, 256, 0, st, (const __nv_bfloat16*)A, lda,
                 (const __nv_bfloat16*)W, N, K, m_total, raw, ld_raw);
  } else {
    dim3 grid((N + 7) / 8, (m_max + 7) / 8);
    if (dtype == RD_DTYPE_FP32)
      launch_pdl(gemm_simt_kernel<float, 8>, grid, 256, 0, st, (const float*)A, lda, (const float*)W, N, K, m_total, raw, ld_raw);
    else
      launch_pdl(gemm_simt_kernel<__nv_bfloat16, 8>, grid, 256, 0, st, (const __nv_bfloat16*)A, lda,
                 (const __nv_bfloat16*)W, N, K, m_total, raw, ld_raw);
  }
  return cudaGetLastError();
}

}  // namespace rd

// Tree-masked attention of the verification forward (Sections 3.3, 3.4).
//
// Row m of sequence b attends the cache slots [0, n_cache[m]) of its sequence and, under tree
// attention, the packed rows j whose bit is set in its mask row; those rows' K/V were written
// to the provisional slots n_cache[m] + j by the rotary kernel, so every key is read from the
// cache.  One CTA per (row, head); each warp walks a strided share of the keys with an online
// softmax and the warps' partial results are merged in shared memory.
#include "rd_internal.cuh"
#include "pdl.cuh"

namespace rd {

constexpr int ATT_WARPS = 4;

template <typename T, int HD>
__global__ void __launch_bounds__(ATT_WARPS * 32) attention_kernel(const float* __restrict__ qkv,
                                                                   const T* __restrict__ kc, const T* __restrict__ vc,
                                                                   T* __restrict__ out, RowTables rt, Dims dm) {
  pdl_enter();
  constexpr int E = HD / 32;  // elements per lane
  __shared__ int32_t tree_slot[1024];
  __shared__ int n_tree_sh;
  __shared__ float sh_m[ATT_WARPS], sh_l[ATT_WARPS], sh_acc[ATT_WARPS][HD];
  const int m = blockIdx.x, h = blockIdx.y;
  if (m >= *rt.m_total) return;
  const int b = rt.seq[m];
  const int n_cache = rt.n_cache[m];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;

  if (threadIdx.x == 0) {
    int cnt = 0;
    if (rt.mask) {
      const uint32_t* mr = rt.mask + ((size_t)b * dm.NMAX + rt.local[m]) * dm.MW;
      for (int wd = 0; wd < dm.MW; ++wd) {
        uint32_t bits = mr[wd];
        while (bits) {
          const int j = __ffs(bits) - 1;
          bits &= bits - 1;
          const int s = n_cache + wd * 32 + j;
          if (s < dm.max_ctx && cnt < 1024) tree_slot[cnt++] = s;
        }
      }
    }
    n_tree_sh = cnt;
  }
  __syncthreads();
  const int n_keys = n_cache + n_tree_sh;

  float q[E];
  const float* qr = qkv + (size_t)m * 3 * dm.d + h * HD;
  const float scale = rsqrtf((float)HD);
#pragma unroll
  for (int e = 0; e < E; ++e) q[e] = qr[lane * E + e] * scale;

  const size_t head_base = ((size_t)b * dm.H + h) * dm.max_ctx * HD;
  float mx = -INFINITY, l = 0.f, acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.f;
  for (int j = w; j < n_keys; j += ATT_WARPS) {
    const int slot = j < n_cache ? j : tree_slot[j - n_cache];
    const T* kp = kc + head_base + (size_t)slot * HD + lane * E;
    const T* vp = vc + head_base + (size_t)slot * HD + lane * E;
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) s = fmaf(q[e], to_f<T>(kp[e]), s);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float nm = fmaxf(mx, s);
    const float corr = __expf(mx - nm), p = __expf(s - nm);
    l = l * corr + p;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = acc[e] * corr + p * to_f<T>(vp[e]);
    mx = nm;
  }
  if (lane == 0) { sh_m[w] = mx; sh_l[w] = l; }
#pragma unroll
  for (int e = 0; e < E; ++e) sh_acc[w][lane * E + e] = acc[e];
  __syncthreads();
  if (w == 0) {
    float gm = -INFINITY;
#pragma unroll
    for (int i = 0; i < ATT_WARPS; ++i) gm = fmaxf(gm, sh_m[i]);
    float gl = 0.f, o[E];
#pragma unroll
    for (int e = 0; e < E; ++e) o[e] = 0.f;
#pragma unroll
    for (int i = 0; i < ATT_WARPS; ++i) {
      const float c = (sh_m[i] == -INFINITY) ? 0.f : __expf(sh_m[i] - gm);
      gl += sh_l[i] * c;
#pragma unroll
      for (int e = 0; e < E; ++e) o[e] += sh_acc[i][lane * E + e] * c;
    }
    const float inv = gl > 0.f ? 1.f / gl : 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) out[(size_t)m * dm.d + h * HD + lane * E + e] = from_f<T>(o[e] * inv);
  }
}

cudaError_t launch_attention(int dtype, const float* qkv, const void* kcache, const void* vcache, void* out_t,
                             const RowTables& rt, const Dims& dm, int m_max, cudaStream_t st) {
  dim3 grid(m_max, dm.H);
#define RD_ATT(T, HD) launch_pdl(attention_kernel<T, HD>, grid, ATT_WARPS * 32, 0, st, qkv, (const T*)kcache, (const T*)vcache, (T*)out_t, rt, dm)
  if (dtype == RD_DTYPE_FP32) {
    if (dm.hd == 64) RD_ATT(float, 64); else if (dm.hd == 128) RD_ATT(float, 128); else return cudaErrorInvalidValue;
  } else {
    if (dm.hd == 64) RD_ATT(__nv_bfloat16, 64); else if (dm.hd == 128) RD_ATT(__nv_bfloat16, 128); else return cudaErrorInvalidValue;
  }
#undef RD_ATT
  return cudaGetLastError();
}

}  // namespace rd

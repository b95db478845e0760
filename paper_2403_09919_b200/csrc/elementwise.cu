// Small row-wise kernels of the verification forward (Section 3.4): embedding gather, RMSNorm,
// rotary embedding + KV-cache write, SwiGLU, row argmax, row tables.  All are bandwidth-trivial
// (activations of at most a few MB that stay in L2); they exist to feed the projections.
#include <cstdlib>
#include "rd_internal.cuh"
#include "gemm_out.cuh"
#include "pdl.cuh"
#include "stage.cuh"

namespace rd {

#define RD_DISPATCH(dtype, ...)                                \
  if ((dtype) == RD_DTYPE_FP32) { using T = float; __VA_ARGS__; } \
  else { using T = __nv_bfloat16; __VA_ARGS__; }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Block-wide sum; every thread gets the result.  blockDim.x multiple of 32, <= 1024.
__device__ __forceinline__ float block_sum(float v, float* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  float t = (lane < nw) ? sh[lane] : 0.f;
  t = warp_sum(t);
  return t;
}

// ---------------------------------------------------------------- embedding gather
template <typename T>
__global__ void embed_kernel(const T* __restrict__ emb, const int32_t* __restrict__ tok, float* __restrict__ x, int d,
                             int V, const int32_t* __restrict__ m_total, int* status) {
  pdl_enter();
  const int m = blockIdx.x;
  if (m >= *m_total) return;
  int t = tok[m];
  if (t < 0 || t >= V) {
    if (threadIdx.x == 0) atomicOr(status, DEV_ERR_TOKEN_RANGE);
    t = min(max(t, 0), V - 1);
  }
  const T* src = emb + (size_t)t * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) x[(size_t)m * d + i] = to_f<T>(src[i]);
}

cudaError_t launch_embed(int dtype, const void* emb, const int32_t* tok, float* x, int d, int V, const int32_t* m_total,
                         int m_max, int* status, cudaStream_t st) {
  RD_DISPATCH(dtype, launch_pdl(embed_kernel<T>, m_max, 256, 0, st, (const T*)emb, tok, x, d, V, m_total, status));
  return cudaGetLastError();
}

// Four consecutive outputs in the activation type (16- or 8-byte store; the address is that much aligned).
__device__ __forceinline__ void store4(float* p, float a, float b, float c, float d) { *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d); }
__device__ __forceinline__ void store4(__nv_bfloat16* p, float a, float b, float c, float d) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 u;
  u.x = *reinterpret_cast<const uint32_t*>(&lo);
  u.y = *reinterpret_cast<const uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = u;
}

// ---------------------------------------------------------------- RMSNorm
// y = x / sqrt(mean(x^2) + eps) * gain, one block per row.  The row is read once with 128-bit loads
// and kept in registers between the reduction and the scaling (d <= 8192).
constexpr int NORM_THREADS = 512;

// Packed gain values of one float4 of the row.
template <typename T> struct Gain4;
template <> struct Gain4<float> {
  float4 g;
  __device__ __forceinline__ void load(const float* p) { g = *reinterpret_cast<const float4*>(p); }
  __device__ __forceinline__ float4 get() const { return g; }
};
template <> struct Gain4<__nv_bfloat16> {
  uint2 g;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { g = *reinterpret_cast<const uint2*>(p); }
  __device__ __forceinline__ float4 get() const {
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&g.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&g.y));
    return make_float4(a.x, a.y, b.x, b.y);
  }
};

// At most 96 registers per thread: one CTA of this kernel (512 threads) and one CTA of the projection that
// follows it then fit the SM's register file together, so the projection is resident and has its first
// weight tiles in flight while the norm still runs.
template <typename T, int NORM_MAXV>
__global__ void __maxnreg__(88)
    rmsnorm_kernel(float* __restrict__ x, GemmOut proj, const T* __restrict__ gain, T* __restrict__ out_t,
                   float* __restrict__ out_f, int d, float eps, const int32_t* __restrict__ m_total, ChainSync cs) {
  chain_begin(cs);
#ifdef RD_PROBE_EMPTY_BODIES   // ceiling probe (a build flag, never in the shipped library): keep the hand-off, drop the work
  chain_wait_cta(cs);
  chain_exit(cs);
  return;
#endif
  __shared__ float sh[32];
  // The first launch of a chain is ordered after everything before it; the later ones may read the row
  // count (written ahead of the chain) before their wait.
  const bool early = cs.signal_ptr != nullptr && cs.wait_ptr != nullptr;
  const int m = blockIdx.x;
  const int nvec = d >> 2;
  // the gain is a weight: requested before the wait, it has arrived when the row has
  Gain4<T> gn[NORM_MAXV];
#pragma unroll
  for (int k = 0; k < NORM_MAXV; ++k) {
    const int i = threadIdx.x + k * NORM_THREADS;
    if (i < nvec) gn[k].load(gain + 4 * i);
  }
  float4* xr = reinterpret_cast<float4*>(x + (size_t)m * d);
  const bool add = proj.raw != nullptr;   // x += the projection that ends the previous block (O or down)
  // Decode-time launches (one row tile, no idle CTA in the projection): every address is worked out while
  // waiting, and the row's loads do not wait for the row count (rows past it exist in memory and are
  // simply not written back).
  // (A launch laid out for several row tiles whose rows fit one after all is a single-tile launch; inside a
  // chain the row count is known up front.)
  int M = early ? *m_total : 0;
  const bool single = proj.m_tiles_max == 1 || (early && M <= proj.mt);
  const bool fast = add && single && (proj.partial == nullptr || proj.all_work);
  const size_t stride = add ? gemm_slot_stride(proj) : 0;
  GemmSrc src[NORM_MAXV];
  if (fast) {
#pragma unroll
    for (int k = 0; k < NORM_MAXV; ++k) {
      const int i = threadIdx.x + k * NORM_THREADS;
      if (i < nvec) { src[k] = gemm_src(proj, GemmRows(1, proj.mt), m, 4 * i); gemm_src_pin(src[k]); }
    }
    asm volatile("" : "+l"(xr));
  }
  chain_wait_cta(cs);
  if (!early) M = *m_total;
  float4 v[NORM_MAXV];
  float ss = 0.f;
  if (fast) {
    GemmData4<5> dat[NORM_MAXV];
    if (m >= M) {
      chain_exit(cs);
      return;
    }
#pragma unroll
    for (int k = 0; k < NORM_MAXV; ++k) {
      const int i = threadIdx.x + k * NORM_THREADS;
      if (i < nvec) { v[k] = __ldcg(xr + i); dat[k] = gemm_load4<5>(src[k], stride); }
    }
#pragma unroll
    for (int k = 0; k < NORM_MAXV; ++k) {
      const int i = threadIdx.x + k * NORM_THREADS;
      if (i < nvec) {
        const float4 q = gemm_sum4(src[k], stride, dat[k]);
        v[k].x += q.x; v[k].y += q.y; v[k].z += q.z; v[k].w += q.w;
        xr[i] = v[k];
        ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
      }
    }
  } else {
    if (m >= M) {
      chain_exit(cs);
      return;
    }
    const GemmRows m_tiles = add ? gemm_m_tiles(proj, M) : GemmRows();
#pragma unroll
    for (int k = 0; k < NORM_MAXV; ++k) {
      const int i = threadIdx.x + k * NORM_THREADS;
      if (i < nvec) {
        v[k] = xr[i];
        if (add) {
          const float4 q = gemm_value4<5>(proj, m_tiles, m, 4 * i);
          v[k].x += q.x; v[k].y += q.y; v[k].z += q.z; v[k].w += q.w;
          xr[i] = v[k];
        }
        ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
      }
    }
  }
  ss = block_sum(ss, sh);
  const float r = rsqrtf(ss / (float)d + eps);
#pragma unroll
  for (int k = 0; k < NORM_MAXV; ++k) {
    const int i = threadIdx.x + k * NORM_THREADS;
    if (i < nvec) {
      const float4 g = gn[k].get();
      const float y0 = v[k].x * r * g.x, y1 = v[k].y * r * g.y, y2 = v[k].z * r * g.z, y3 = v[k].w * r * g.w;
      const size_t o = (size_t)m * d + 4 * i;
      if (out_t) store4(out_t + o, y0, y1, y2, y3);
      if (out_f) *reinterpret_cast<float4*>(out_f + o) = make_float4(y0, y1, y2, y3);
    }
  }
  chain_exit(cs);
}


// Launches of more than one row tile (prompts, wide beams, large batches).  The kernels above are built around the
// latency of a single short pass per CTA; with thousands of rows that becomes wave after wave of CTAs that each pay
// the hand-off poll, the row-count load and one round trip for their data.  The *_wide variants fill the SMs once
// and walk the rows in a loop, every load of a row in flight before the first is used.
// The row-loop variants take over where the host-side bound on the rows exceeds one row tile (measured at bounds of
// 330 rows, 170-220 rows present: 2-5 % of the step against the kernels above; at a bound of 164 rows they lose).
// RD_WIDE_MIN: tuning toggle.
static const int WIDE_ROWS_MIN = getenv("RD_WIDE_MIN") ? atoi(getenv("RD_WIDE_MIN")) : 256;
static int wide_sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}
// Partial slots loaded up front (a longer list takes the tail loop).  With more (tile pair, row tile) groups than CTAs a
// tile is cut at most once: gate|up always, QKV mostly; O and down have few tiles, cut among several CTAs each.
constexpr int WIDE_FOLD_NORM = 2, WIDE_FOLD_ROPE = 2, WIDE_FOLD_SWIGLU = 1;

template <typename T, int NORM_MAXV>
__global__ void __launch_bounds__(NORM_THREADS, NORM_MAXV <= 2 ? 2 : 1)
    rmsnorm_wide_kernel(float* __restrict__ x, GemmOut proj, const T* __restrict__ gain, T* __restrict__ out_t,
                        float* __restrict__ out_f, int d, float eps, const int32_t* __restrict__ m_total, ChainSync cs) {
  chain_begin(cs);
  __shared__ float sh[32];
  // inside a chain (but not as its first launch) the row count, written ahead of the chain, may be read before the wait
  const bool early = cs.signal_ptr != nullptr && cs.wait_ptr != nullptr;
  int M = early ? *m_total : 0;
  chain_wait_cta(cs);
  if (!early) M = *m_total;
  const int nvec = d >> 2;
  const bool add = proj.raw != nullptr;   // x += the projection that ends the previous block (O or down)
  const GemmRows m_tiles = add ? gemm_m_tiles(proj, M) : GemmRows();
  for (int m = blockIdx.x; m < M; m += gridDim.x) {
    float4* xr = reinterpret_cast<float4*>(x + (size_t)m * d);
    float4 v[NORM_MAXV];
    GemmPending4<WIDE_FOLD_NORM> pd[NORM_MAXV];
#pragma unroll
    for (int k = 0; k < NORM_MAXV; ++k) {
      const int i = threadIdx.x + k * NORM_THREADS;
      if (i < nvec) {
        v[k] = __ldcg(xr + i);
        if (add) pd[k] = gemm_issue4<WIDE_FOLD_NORM>(proj, m_tiles, m, 4 * i);
      }
    }
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < NORM_MAXV; ++k) {
      const int i = threadIdx.x + k * NORM_THREADS;
      if (i < nvec) {
        if (add) {
          const float4 q = gemm_finish4(proj, m_tiles, pd[k]);
          v[k].x += q.x; v[k].y += q.y; v[k].z += q.z; v[k].w += q.w;
          xr[i] = v[k];
        }
        ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
      }
    }
    ss = block_sum(ss, sh);
    const float r = rsqrtf(ss / (float)d + eps);
#pragma unroll
    for (int k = 0; k < NORM_MAXV; ++k) {
      const int i = threadIdx.x + k * NORM_THREADS;
      if (i < nvec) {
        Gain4<T> gn;
        gn.load(gain + 4 * i);
        const float4 g = gn.get();
        const float y0 = v[k].x * r * g.x, y1 = v[k].y * r * g.y, y2 = v[k].z * r * g.z, y3 = v[k].w * r * g.w;
        const size_t o = (size_t)m * d + 4 * i;
        if (out_t) store4(out_t + o, y0, y1, y2, y3);
        if (out_f) *reinterpret_cast<float4*>(out_f + o) = make_float4(y0, y1, y2, y3);
      }
    }
  }
  chain_exit(cs);
}

// x: residual stream (updated in place when proj != nullptr: x += proj).
cudaError_t launch_rmsnorm(int dtype, float* x, const GemmOut* proj, const void* gain, void* out_t, float* out_f32, int d,
                           float eps, const int32_t* m_total, int m_max, Chain* chain, cudaStream_t st) {
  if (d > 4 * NORM_THREADS * 4 || (d & 3)) return cudaErrorInvalidValue;
  GemmOut g{};
  if (proj) g = *proj;
  // the first launch of a chain starts after everything before it has completed (see launch_ordered)
  const bool first = chain && chain->enabled && chain->prev_ptr == nullptr;
  if (m_max > WIDE_ROWS_MIN) {   // several row tiles
    const int per_sm = (d <= 4 * NORM_THREADS * 2) ? 2 : 1;   // resident CTAs per SM: one wave walks all rows
    const int grid = m_max < per_sm * wide_sm_count() ? m_max : per_sm * wide_sm_count();
    const ChainSync cs = chain ? chain->link((unsigned)grid, true) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
#define RD_NORM_WIDE(MAXV)                                                                                                \
  RD_DISPATCH(dtype, if (first) launch_ordered(rmsnorm_wide_kernel<T, MAXV>, grid, NORM_THREADS, 0, st, x, g, (const T*)gain, \
                                               (T*)out_t, out_f32, d, eps, m_total, cs);                                  \
              else launch_pdl(rmsnorm_wide_kernel<T, MAXV>, grid, NORM_THREADS, 0, st, x, g, (const T*)gain, (T*)out_t,    \
                              out_f32, d, eps, m_total, cs))
    if (d <= 4 * NORM_THREADS * 2) {
      RD_NORM_WIDE(2);
    } else {
      RD_NORM_WIDE(4);
    }
#undef RD_NORM_WIDE
    return cudaGetLastError();
  }
  const ChainSync cs = chain ? chain->link((unsigned)m_max, true) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
#define RD_NORM_LAUNCH(MAXV)                                                                                              \
  RD_DISPATCH(dtype, if (first) launch_ordered(rmsnorm_kernel<T, MAXV>, m_max, NORM_THREADS, 0, st, x, g, (const T*)gain,  \
                                               (T*)out_t, out_f32, d, eps, m_total, cs);                                  \
              else launch_pdl(rmsnorm_kernel<T, MAXV>, m_max, NORM_THREADS, 0, st, x, g, (const T*)gain, (T*)out_t,        \
                              out_f32, d, eps, m_total, cs))
  if (d <= 4 * NORM_THREADS * 2) {
    RD_NORM_LAUNCH(2);
  } else {
    RD_NORM_LAUNCH(4);
  }
#undef RD_NORM_LAUNCH
  return cudaGetLastError();
}

// ---------------------------------------------------------------- rotary table
// cos/sin of pos * theta^(-2i/hd) for every row of the pass, computed once per forward (all layers
// share it).  The angle is formed in double: positions reach several thousand and its rounding
// error in single precision would scale with them.
__global__ void rope_table_kernel(const int32_t* __restrict__ pos, float2* __restrict__ table, int half, float theta,
                                  const int32_t* __restrict__ m_total) {
  pdl_enter();
  const int m = blockIdx.x;
  if (m >= *m_total) return;
  const double l2t = log2((double)theta);
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    const double ang = (double)pos[m] * exp2(-((double)i / half) * l2t);
    double sd, cd;
    sincos(ang, &sd, &cd);
    table[(size_t)m * half + i] = make_float2((float)cd, (float)sd);
  }
}

cudaError_t launch_rope_table(const int32_t* pos, float* table, int hd, float theta, const int32_t* m_total, int m_max,
                              cudaStream_t st) {
  launch_pdl(rope_table_kernel, m_max, 64, 0, st, pos, reinterpret_cast<float2*>(table), hd / 2, theta, m_total);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- rotary embedding + KV write
// qkv: [M][3d] fp32 (Q | K | V).  Q is rotated in place; rotated K and V go to the cache slot of
// the row.  Pairing (i, i + hd/2).
// One thread per pair of adjacent rotary indices (i, i+1) of one head: it reads Q, K, V at columns i, i+1
// and i+hd/2, i+hd/2+1 (one tile of the projection, one fold), all in a single batch of loads issued right
// after the wait, together with the row's table entries -- one L2 round trip for the whole kernel.
// What bounds the kernel is how fast ONE SM can pull its share out of the L2 (a few tens of GB/s), so the
// rows are spread over as many SMs as possible: 256-thread CTAs, several per row, at no more than 88
// registers so that they are all resident beside the projection that runs before them.
constexpr int ROPE_THREADS = 256;
constexpr int ROPE_FOLD = 4;   // partial slots loaded up front: a QKV tile (64+ k-blocks) is rarely cut in more than three

__device__ __forceinline__ void store2(float* p, float a, float b) { *reinterpret_cast<float2*>(p) = make_float2(a, b); }
__device__ __forceinline__ void store2(__nv_bfloat16* p, float a, float b) {
  *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(a, b);
}

template <typename T>
__global__ void __maxnreg__(88) rope_kv_kernel(float* __restrict__ qkv, GemmOut proj, T* __restrict__ kc, T* __restrict__ vc,
                                               const float2* __restrict__ table, RowTables rt, Dims dm, int* status,
                                               ChainSync cs) {
  chain_begin(cs);
#ifdef RD_PROBE_EMPTY_BODIES   // ceiling probe (a build flag, never in the shipped library): keep the hand-off, drop the work
  chain_wait_cta(cs);
  chain_exit(cs);
  return;
#endif
  // inside a chain the row tables and the rotary table (written ahead of the chain) may be read before the wait
  const bool early = cs.signal_ptr != nullptr;
  if (!early) chain_wait_cta(cs);
  const int m = blockIdx.x;
  const int d = dm.d, hd = dm.hd, half = hd >> 1;
  const int n_items = dm.H * (half >> 1);
  const int idx = blockIdx.y * ROPE_THREADS + threadIdx.x;   // the grid covers every item of the row once
  const bool active = idx < n_items;
  const int h = idx / (half >> 1), i = (idx - h * (half >> 1)) * 2;
  const int o = h * hd + i;
  float* row = qkv + (size_t)m * 3 * d;
  // decode-time launches (one row tile, no idle CTA in the projection): every address is known before the
  // projection has produced anything
  const bool single = proj.m_tiles_max == 1 || (early && *rt.m_total <= proj.mt);   // rows that fit one row tile after all
  const bool fast = single && (proj.partial == nullptr || proj.all_work);
  GemmSrc sq, sk, sv;
  const size_t stride = gemm_slot_stride(proj);
  const float2* tab = table + (size_t)m * half + i;
  if (fast && active) {
    sq = gemm_src(proj, GemmRows(1, proj.mt), m, o); sk = gemm_src(proj, GemmRows(1, proj.mt), m, d + o); sv = gemm_src(proj, GemmRows(1, proj.mt), m, 2 * d + o);
    gemm_src_pin(sq); gemm_src_pin(sk); gemm_src_pin(sv);
    asm volatile("" : "+l"(tab), "+l"(row));
  }
  int M = 0, b = 0, slot = 0;
  float4 cs2 = make_float4(0.f, 0.f, 0.f, 0.f);   // (cos, sin) of i and i+1
  if (fast && active) {
    M = *rt.m_total; b = rt.seq[m]; slot = rt.slot[m];
    cs2 = *reinterpret_cast<const float4*>(tab);
  }
  if (early) chain_wait_cta(cs);
  if (fast) {
    if (active && m < M) {
      // one batch of loads, then the arithmetic
      const auto dq1 = gemm_load2<ROPE_FOLD>(sq, stride), dq2 = gemm_load2<ROPE_FOLD>(sq, stride, half);
      const auto dk1 = gemm_load2<ROPE_FOLD>(sk, stride), dk2 = gemm_load2<ROPE_FOLD>(sk, stride, half);
      const auto dv1 = gemm_load2<ROPE_FOLD>(sv, stride), dv2 = gemm_load2<ROPE_FOLD>(sv, stride, half);
      {
        const bool slot_ok = slot >= 0 && slot < dm.max_ctx;
        if (!slot_ok && idx == 0) atomicOr(status, DEV_ERR_CAPACITY);
        const float2 q1 = gemm_sum2(sq, stride, dq1), q2 = gemm_sum2(sq, stride, dq2, half);
        const float2 k1 = gemm_sum2(sk, stride, dk1), k2 = gemm_sum2(sk, stride, dk2, half);
        const float2 v1 = gemm_sum2(sv, stride, dv1), v2 = gemm_sum2(sv, stride, dv2, half);
        // the attention kernel reads the rotated Q from the projection's own buffer
        store2(row + o, q1.x * cs2.x - q2.x * cs2.y, q1.y * cs2.z - q2.y * cs2.w);
        store2(row + o + half, q2.x * cs2.x + q1.x * cs2.y, q2.y * cs2.z + q1.y * cs2.w);
        if (slot_ok) {
          const size_t base = (((size_t)b * dm.H + h) * dm.max_ctx + slot) * hd + i;
          store2(kc + base, k1.x * cs2.x - k2.x * cs2.y, k1.y * cs2.z - k2.y * cs2.w);
          store2(kc + base + half, k2.x * cs2.x + k1.x * cs2.y, k2.y * cs2.z + k1.y * cs2.w);
          store2(vc + base, v1.x, v1.y);
          store2(vc + base + half, v2.x, v2.y);
        }
      }
    }
  } else {
    // prompt-sized launches (several row tiles) and projections shorter than the grid
    M = *rt.m_total;
    if (m < M && active) {
      const GemmRows m_tiles = gemm_m_tiles(proj, M);
      b = rt.seq[m]; slot = rt.slot[m];
      const bool slot_ok = slot >= 0 && slot < dm.max_ctx;
      if (!slot_ok && idx == 0) atomicOr(status, DEV_ERR_CAPACITY);
      cs2 = *reinterpret_cast<const float4*>(tab);
      const GemmFold fq = gemm_fold_or_none(proj, m_tiles, m, o), fk = gemm_fold_or_none(proj, m_tiles, m, d + o),
                     fv = gemm_fold_or_none(proj, m_tiles, m, 2 * d + o);
      const auto pq1 = gemm_issue2<ROPE_FOLD>(proj, m_tiles, fq, m, o, 0), pq2 = gemm_issue2<ROPE_FOLD>(proj, m_tiles, fq, m, o + half, half);
      const auto pk1 = gemm_issue2<ROPE_FOLD>(proj, m_tiles, fk, m, d + o, 0), pk2 = gemm_issue2<ROPE_FOLD>(proj, m_tiles, fk, m, d + o + half, half);
      const auto pv1 = gemm_issue2<ROPE_FOLD>(proj, m_tiles, fv, m, 2 * d + o, 0), pv2 = gemm_issue2<ROPE_FOLD>(proj, m_tiles, fv, m, 2 * d + o + half, half);
      const float2 q1 = gemm_finish2(proj, m_tiles, fq, 0, pq1), q2 = gemm_finish2(proj, m_tiles, fq, half, pq2);
      const float2 k1 = gemm_finish2(proj, m_tiles, fk, 0, pk1), k2 = gemm_finish2(proj, m_tiles, fk, half, pk2);
      const float2 v1 = gemm_finish2(proj, m_tiles, fv, 0, pv1), v2 = gemm_finish2(proj, m_tiles, fv, half, pv2);
      store2(row + o, q1.x * cs2.x - q2.x * cs2.y, q1.y * cs2.z - q2.y * cs2.w);
      store2(row + o + half, q2.x * cs2.x + q1.x * cs2.y, q2.y * cs2.z + q1.y * cs2.w);
      if (slot_ok) {
        const size_t base = (((size_t)b * dm.H + h) * dm.max_ctx + slot) * hd + i;
        store2(kc + base, k1.x * cs2.x - k2.x * cs2.y, k1.y * cs2.z - k2.y * cs2.w);
        store2(kc + base + half, k2.x * cs2.x + k1.x * cs2.y, k2.y * cs2.z + k1.y * cs2.w);
        store2(vc + base, v1.x, v1.y);
        store2(vc + base + half, v2.x, v2.y);
      }
    }
  }
  chain_exit(cs);
}


// Many rows: blockIdx.x picks a group of heads (ROPW_COLS columns), blockIdx.y a contiguous run of rows.  The Q, K
// and V segments of a row (contiguous, ROPW_COLS x 4 bytes each) come in through a ring of shared-memory stages filled
// by thread 0 with bulk asynchronous copies, ROPW_STAGES - 1 rows ahead (stage.cuh; see swiglu_wide_kernel).  Partial
// sums of tiles cut between CTAs are added from global memory by the threads whose columns they concern.
constexpr int ROPW_THREADS = 256;
constexpr int ROPW_COLS = 1024;     // one item (two adjacent dimensions and their partners half a head on) per thread
constexpr int ROPW_STAGES = 3;      // 3 x 3 x 4 KB per CTA (static shared memory)
template <typename T>
__global__ void __launch_bounds__(ROPW_THREADS, 4)
    rope_kv_wide_kernel(float* __restrict__ qkv, GemmOut proj, T* __restrict__ kc, T* __restrict__ vc,
                        const float2* __restrict__ table, RowTables rt, Dims dm, int* status, ChainSync cs) {
  chain_begin(cs);
  __shared__ __align__(128) float ring[ROPW_STAGES][3][ROPW_COLS];   // 36 KB
  __shared__ __align__(8) unsigned long long bars[ROPW_STAGES];
  const uint32_t ring_u = stage_smem_u32(ring), bars_u = stage_smem_u32(bars);
  if (threadIdx.x == 0) {
    for (int s = 0; s < ROPW_STAGES; ++s) stage_bar_init(bars_u + 8u * s, 1);
    stage_bar_init_fence();
  }
  const int d = dm.d, hd = dm.hd, half = hd >> 1;
  const int heads_per_cta = ROPW_COLS / hd;
  const int h0 = blockIdx.x * heads_per_cta;
  const int n_heads = min(heads_per_cta, dm.H - h0);
  const int c0 = h0 * hd, ncol = n_heads * hd;           // this CTA's columns inside each of Q, K, V
  const uint32_t seg_bytes = (uint32_t)ncol * 4u;
  const int hl = threadIdx.x / (half >> 1), i = (threadIdx.x - hl * (half >> 1)) * 2;   // head inside the group, dimension
  const bool active = hl < n_heads;
  const int j = hl * hd + i;                              // column inside the segment
  const int h = h0 + hl, o = c0 + j;
  // inside a chain the row count, written ahead of the chain, may be read before the wait
  const bool early = cs.signal_ptr != nullptr && cs.wait_ptr != nullptr;
  int M = early ? *rt.m_total : 0;
  chain_wait_cta(cs);   // (its barrier also publishes the initialised mbarriers)
  if (!early) M = *rt.m_total;
  const GemmRows m_tiles = gemm_m_tiles(proj, M);
  const int m_begin = gemm_rows_begin(M, gridDim.y, blockIdx.y), m_end = gemm_rows_begin(M, gridDim.y, blockIdx.y + 1);
  const int n_rows = m_end - m_begin;
  auto issue = [&](int r) {   // thread 0: row m_begin + r into slot r % ROPW_STAGES
    const int s = r % ROPW_STAGES;
    const float* src = qkv + (size_t)(m_begin + r) * 3 * d + c0;
    stage_expect_tx(bars_u + 8u * s, 3u * seg_bytes);
#pragma unroll
    for (int part = 0; part < 3; ++part)
      stage_copy(ring_u + (uint32_t)((s * 3 + part) * ROPW_COLS) * 4u, src + (size_t)part * d, seg_bytes, bars_u + 8u * s);
  };
  if (threadIdx.x == 0) {
    chain_fence_async_reads();   // the projection wrote its output with ordinary stores
    for (int r = 0; r < ROPW_STAGES - 1 && r < n_rows; ++r) issue(r);
  }
  const bool cut_any = proj.partial != nullptr;
  const size_t slot_stride = gemm_slot_stride(proj);
  int tile_end = 0, cur_tile = 0;
  GemmFold f3[3];          // folds of this thread's Q, K and V columns: they change only from one row tile to the next
  bool cut = false;
  uint32_t s = 0, ph = 0;
  for (int r = 0; r < n_rows; ++r) {
    const int m = m_begin + r;
    if (threadIdx.x == 0 && r + ROPW_STAGES - 1 < n_rows) issue(r + ROPW_STAGES - 1);   // slot released by the last barrier
    int b = 0, slot = -1;
    float4 cs2 = make_float4(0.f, 0.f, 0.f, 0.f);   // (cos, sin) of i and i+1
    if (active) {
      b = rt.seq[m]; slot = rt.slot[m];
      cs2 = *reinterpret_cast<const float4*>(table + (size_t)m * half + i);
      if (cut_any && m >= tile_end) {
        cur_tile = m / m_tiles.rows;
        tile_end = (cur_tile + 1) * m_tiles.rows;
        cut = false;
#pragma unroll
        for (int part = 0; part < 3; ++part) {
          f3[part] = gemm_fold(proj, m_tiles, cur_tile * m_tiles.rows, part * d + o);
          cut = cut || f3[part].c_next <= f3[part].c_last;
        }
      }
    }
    stage_wait(bars_u + 8u * s, ph, status, DEV_ERR_TIMEOUT);
    if (active) {
      float2 v1[3], v2[3];   // (i, i+1) and (i + half, i + half + 1) of Q, K, V
#pragma unroll
      for (int part = 0; part < 3; ++part) {
        v1[part] = *reinterpret_cast<const float2*>(&ring[s][part][j]);
        v2[part] = *reinterpret_cast<const float2*>(&ring[s][part][j + half]);
      }
      if (cut) {   // add the other contributors' sums in CTA order
        const size_t doff = (size_t)(m - cur_tile * m_tiles.rows) * 128;
#pragma unroll
        for (int part = 0; part < 3; ++part)
          for (int c = f3[part].c_next; c <= f3[part].c_last; ++c)
            if (gemm_has_work(proj, m_tiles, c)) {
              const float* pp = proj.partial + (size_t)c * slot_stride + f3[part].off + doff;
              const float2 t1 = __ldcg(reinterpret_cast<const float2*>(pp)), t2 = __ldcg(reinterpret_cast<const float2*>(pp + half));
              v1[part].x += t1.x; v1[part].y += t1.y; v2[part].x += t2.x; v2[part].y += t2.y;
            }
      }
      const bool slot_ok = slot >= 0 && slot < dm.max_ctx;
      if (!slot_ok && i == 0 && h == 0) atomicOr(status, DEV_ERR_CAPACITY);
      // the attention kernel reads the rotated Q from the projection's own buffer
      float* row = qkv + (size_t)m * 3 * d;
      store2(row + o, v1[0].x * cs2.x - v2[0].x * cs2.y, v1[0].y * cs2.z - v2[0].y * cs2.w);
      store2(row + o + half, v2[0].x * cs2.x + v1[0].x * cs2.y, v2[0].y * cs2.z + v1[0].y * cs2.w);
      if (slot_ok) {
        const size_t base = (((size_t)b * dm.H + h) * dm.max_ctx + slot) * hd + i;
        store2(kc + base, v1[1].x * cs2.x - v2[1].x * cs2.y, v1[1].y * cs2.z - v2[1].y * cs2.w);
        store2(kc + base + half, v2[1].x * cs2.x + v1[1].x * cs2.y, v2[1].y * cs2.z + v1[1].y * cs2.w);
        store2(vc + base, v1[2].x, v1[2].y);
        store2(vc + base + half, v2[2].x, v2[2].y);
      }
    }
    __syncthreads();   // every thread is done with the slot
    if (++s == ROPW_STAGES) { s = 0; ph ^= 1u; }
  }
  chain_exit(cs);
}

cudaError_t launch_rope_kv(int dtype, float* qkv, const GemmOut& proj, void* kcache, void* vcache, const float* table,
                           const RowTables& rt, const Dims& dm, int m_max, int* status, Chain* chain, cudaStream_t st) {
  const int n_items = dm.H * (dm.hd / 4);
  dim3 grid(m_max, (n_items + ROPE_THREADS - 1) / ROPE_THREADS);
  if (m_max > WIDE_ROWS_MIN && ROPW_COLS % dm.hd == 0 && (ROPW_COLS / dm.hd) * (dm.hd / 4) <= ROPW_THREADS) {
    // several row tiles: four CTAs per SM (36 KB of stages each) walk the rows
    const int heads_per_cta = ROPW_COLS / dm.hd;
    dim3 gw((dm.H + heads_per_cta - 1) / heads_per_cta, 1);
    const int gy = (4 * wide_sm_count() + (int)gw.x - 1) / (int)gw.x;
    gw.y = gy < m_max ? gy : m_max;
    const ChainSync cs = chain ? chain->link(gw.x * gw.y, true) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
    RD_DISPATCH(dtype, launch_pdl(rope_kv_wide_kernel<T>, gw, ROPW_THREADS, 0, st, qkv, proj, (T*)kcache, (T*)vcache,
                                  reinterpret_cast<const float2*>(table), rt, dm, status, cs));
    return cudaGetLastError();
  }
  const ChainSync cs = chain ? chain->link(grid.x * grid.y, true) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
  RD_DISPATCH(dtype, launch_pdl(rope_kv_kernel<T>, grid, ROPE_THREADS, 0, st, qkv, proj, (T*)kcache, (T*)vcache,
                                reinterpret_cast<const float2*>(table), rt, dm, status, cs));
  return cudaGetLastError();
}

// ---------------------------------------------------------------- SwiGLU
// Two float4 items of the row per thread, every load of both issued before either is used.  Small CTAs
// (128 threads), many per row: the kernel is bounded by the rate at which one SM pulls data out of the L2,
// so the work is spread evenly over all SMs; at 88 registers they are all resident beside the gate|up
// projection.
constexpr int SWIGLU_THREADS = 128;
constexpr int SWIGLU_ITEMS = 2;
constexpr int SWIGLU_FOLD = 2;  // a gate|up tile is cut between two CTAs at most once the stream is longer than a tile per CTA

template <typename T>
__global__ void __maxnreg__(88) swiglu_kernel(GemmOut proj, T* __restrict__ out, int F, const int32_t* __restrict__ m_total,
                                              ChainSync cs) {
  chain_begin(cs);
#ifdef RD_PROBE_EMPTY_BODIES   // ceiling probe (a build flag, never in the shipped library): keep the hand-off, drop the work
  chain_wait_cta(cs);
  chain_exit(cs);
  return;
#endif
  const bool early = cs.signal_ptr != nullptr;   // inside a chain the row count (written ahead of it) may be read now
  if (!early) chain_wait_cta(cs);
  const int m = blockIdx.y;
  const size_t stride = gemm_slot_stride(proj);
  const int M = *m_total;
  const bool single = proj.m_tiles_max == 1 || M <= proj.mt;   // rows that fit one row tile after all
  const bool fast = single && (proj.partial == nullptr || proj.all_work);
  GemmSrc sg[SWIGLU_ITEMS], su[SWIGLU_ITEMS];
  T* dst[SWIGLU_ITEMS];
  bool act[SWIGLU_ITEMS];
#pragma unroll
  for (int k = 0; k < SWIGLU_ITEMS; ++k) {
    const int f = ((blockIdx.x * SWIGLU_ITEMS + k) * SWIGLU_THREADS + threadIdx.x) * 4;
    act[k] = f < F;
    dst[k] = out + (size_t)m * F + f;
    if (fast && act[k]) {
      sg[k] = gemm_src(proj, GemmRows(1, proj.mt), m, f); su[k] = gemm_src(proj, GemmRows(1, proj.mt), m, F + f);
      gemm_src_pin(sg[k]); gemm_src_pin(su[k]);
      asm volatile("" : "+l"(dst[k]));
    }
  }
  if (early) chain_wait_cta(cs);
  if (fast) {
    if (m < M) {
      GemmData4<SWIGLU_FOLD> dg[SWIGLU_ITEMS], du[SWIGLU_ITEMS];
#pragma unroll
      for (int k = 0; k < SWIGLU_ITEMS; ++k)
        if (act[k]) { dg[k] = gemm_load4<SWIGLU_FOLD>(sg[k], stride); du[k] = gemm_load4<SWIGLU_FOLD>(su[k], stride); }
#pragma unroll
      for (int k = 0; k < SWIGLU_ITEMS; ++k)
        if (act[k]) {
          const float4 g = gemm_sum4(sg[k], stride, dg[k]), u = gemm_sum4(su[k], stride, du[k]);
          store4(dst[k], silu_f(g.x) * u.x, silu_f(g.y) * u.y, silu_f(g.z) * u.z, silu_f(g.w) * u.w);
        }
    }
  } else {
    if (m < M) {
      const GemmRows m_tiles = gemm_m_tiles(proj, M);
      for (int k = 0; k < SWIGLU_ITEMS; ++k) {
        const int f = ((blockIdx.x * SWIGLU_ITEMS + k) * SWIGLU_THREADS + threadIdx.x) * 4;
        if (f < F) {
          const float4 g = gemm_value4<SWIGLU_FOLD>(proj, m_tiles, m, f), u = gemm_value4<SWIGLU_FOLD>(proj, m_tiles, m, F + f);
          store4(dst[k], silu_f(g.x) * u.x, silu_f(g.y) * u.y, silu_f(g.z) * u.z, silu_f(g.w) * u.w);
        }
      }
    }
  }
  chain_exit(cs);
}


// Many rows: blockIdx.x picks SWS_COLS consecutive columns, blockIdx.y a contiguous run of rows.  The gate and the up
// segment of a row (SWS_COLS x 4 bytes each, contiguous) come in through a ring of shared-memory stages filled by
// thread 0 with bulk asynchronous copies, SWS_STAGES - 1 rows ahead of the row being worked on (stage.cuh), so what
// the CTA has in flight does not depend on its registers.  Partial sums (with far more tiles than CTAs a tile is cut at
// most once, and about one tile in five is) are added from global memory by the threads whose columns they concern.
constexpr int SWS_THREADS = 256;
constexpr int SWS_COLS = 2048;      // two float4 per thread
constexpr int SWS_STAGES = 4;       // 4 x (8 + 8) KB per CTA
template <typename T>
__global__ void __launch_bounds__(SWS_THREADS, 3)
    swiglu_wide_kernel(GemmOut proj, T* __restrict__ out, int F, const int32_t* __restrict__ m_total, int32_t* status,
                       ChainSync cs) {
  chain_begin(cs);
  extern __shared__ __align__(128) uint8_t sws_smem[];
  __shared__ __align__(8) unsigned long long sws_bars[SWS_STAGES];
  float* ring = reinterpret_cast<float*>(sws_smem);   // [SWS_STAGES][gate | up][SWS_COLS]
  const uint32_t ring_u = stage_smem_u32(ring), bars_u = stage_smem_u32(sws_bars);
  if (threadIdx.x == 0) {
    for (int s = 0; s < SWS_STAGES; ++s) stage_bar_init(bars_u + 8u * s, 1);
    stage_bar_init_fence();
  }
  // inside a chain the row count, written ahead of the chain, may be read before the wait
  const bool early = cs.signal_ptr != nullptr && cs.wait_ptr != nullptr;
  int M = early ? *m_total : 0;
  chain_wait_cta(cs);   // (its barrier also publishes the initialised mbarriers)
  if (!early) M = *m_total;
  const GemmRows m_tiles = gemm_m_tiles(proj, M);
  const int c0 = blockIdx.x * SWS_COLS;
  const int ncol = min(SWS_COLS, F - c0);
  const uint32_t seg_bytes = (uint32_t)ncol * 4u;
  const int m_begin = gemm_rows_begin(M, gridDim.y, blockIdx.y), m_end = gemm_rows_begin(M, gridDim.y, blockIdx.y + 1);
  const int n_rows = m_end - m_begin;
  auto issue = [&](int i) {   // thread 0: row m_begin + i into slot i % SWS_STAGES
    const int s = i % SWS_STAGES;
    const float* src = proj.raw + (size_t)(m_begin + i) * proj.ld + c0;
    stage_expect_tx(bars_u + 8u * s, 2u * seg_bytes);
    stage_copy(ring_u + (uint32_t)(s * 2) * SWS_COLS * 4u, src, seg_bytes, bars_u + 8u * s);
    stage_copy(ring_u + (uint32_t)(s * 2 + 1) * SWS_COLS * 4u, src + F, seg_bytes, bars_u + 8u * s);
  };
  if (threadIdx.x == 0) {
    chain_fence_async_reads();   // the projection wrote its output with ordinary stores
    for (int i = 0; i < SWS_STAGES - 1 && i < n_rows; ++i) issue(i);
  }
  const int j0 = threadIdx.x * 4, j1 = j0 + SWS_THREADS * 4;   // this thread's two float4 inside the segment
  const bool cut_any = proj.partial != nullptr;
  int tile_end = 0, cur_tile = 0;
  const size_t slot = gemm_slot_stride(proj);
  GemmFold fg[2], fu[2];   // the fold of a column changes only from one row tile to the next
  bool cut[2] = {false, false};
  uint32_t s = 0, ph = 0;
  for (int i = 0; i < n_rows; ++i) {
    const int m = m_begin + i;
    if (threadIdx.x == 0 && i + SWS_STAGES - 1 < n_rows) issue(i + SWS_STAGES - 1);   // slot released by the last barrier
    if (cut_any && m >= tile_end) {
      cur_tile = m / m_tiles.rows;
      tile_end = (cur_tile + 1) * m_tiles.rows;
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int j = k ? j1 : j0;
        if (j < ncol) {
          fg[k] = gemm_fold(proj, m_tiles, cur_tile * m_tiles.rows, c0 + j);
          fu[k] = gemm_fold(proj, m_tiles, cur_tile * m_tiles.rows, F + c0 + j);
          cut[k] = fg[k].c_next <= fg[k].c_last || fu[k].c_next <= fu[k].c_last;
        }
      }
    }
    stage_wait(bars_u + 8u * s, ph, status, DEV_ERR_TIMEOUT);
    const float* sg = ring + (size_t)(s * 2) * SWS_COLS;
    const float* su = sg + SWS_COLS;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int j = k ? j1 : j0;
      if (j < ncol) {
        float4 g = *reinterpret_cast<const float4*>(sg + j), u = *reinterpret_cast<const float4*>(su + j);
        if (cut[k]) {   // add the other contributors' sums in CTA order
          const size_t doff = (size_t)(m - cur_tile * m_tiles.rows) * 128;
          for (int c = fg[k].c_next; c <= fg[k].c_last; ++c)
            if (gemm_has_work(proj, m_tiles, c)) {
              const float4 t = __ldcg(reinterpret_cast<const float4*>(proj.partial + (size_t)c * slot + fg[k].off + doff));
              g.x += t.x; g.y += t.y; g.z += t.z; g.w += t.w;
            }
          for (int c = fu[k].c_next; c <= fu[k].c_last; ++c)
            if (gemm_has_work(proj, m_tiles, c)) {
              const float4 t = __ldcg(reinterpret_cast<const float4*>(proj.partial + (size_t)c * slot + fu[k].off + doff));
              u.x += t.x; u.y += t.y; u.z += t.z; u.w += t.w;
            }
        }
        store4(out + (size_t)m * F + c0 + j, silu_f(g.x) * u.x, silu_f(g.y) * u.y, silu_f(g.z) * u.z, silu_f(g.w) * u.w);
      }
    }
    __syncthreads();   // every thread is done with the slot
    if (++s == SWS_STAGES) { s = 0; ph ^= 1u; }
  }
  chain_exit(cs);
}

// Once per handle (and so per device): opt-in of the kernels that take more than 48 KB of dynamic shared memory.
cudaError_t elementwise_prepare(int dtype) {
  cudaError_t e = cudaErrorInvalidValue;
  const int smem = SWS_STAGES * 2 * SWS_COLS * (int)sizeof(float);
  RD_DISPATCH(dtype, e = cudaFuncSetAttribute(swiglu_wide_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  return e;
}

// proj: the gate|up projection [M][2F]; out: [M][F].  F must be a multiple of 4.
cudaError_t launch_swiglu(int dtype, const GemmOut& proj, void* out_t, int F, const int32_t* m_total, int m_max,
                          int32_t* status, Chain* chain, cudaStream_t st) {
  const int per_cta = SWIGLU_THREADS * SWIGLU_ITEMS * 4;
  dim3 grid((F + per_cta - 1) / per_cta, m_max);
  if (m_max > WIDE_ROWS_MIN) {   // several row tiles: three CTAs per SM (64 KB of stages each) walk the rows
    const size_t smem = (size_t)SWS_STAGES * 2 * SWS_COLS * sizeof(float);   // opted in by elementwise_prepare
    grid.x = (F + SWS_COLS - 1) / SWS_COLS;
    const int gy = (3 * wide_sm_count() + (int)grid.x - 1) / (int)grid.x;
    grid.y = gy < m_max ? gy : m_max;
    const ChainSync cs = chain ? chain->link(grid.x * grid.y, true) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
    RD_DISPATCH(dtype, launch_pdl(swiglu_wide_kernel<T>, grid, SWS_THREADS, smem, st, proj, (T*)out_t, F, m_total, status, cs));
    return cudaGetLastError();
  }
  const ChainSync cs = chain ? chain->link(grid.x * grid.y, true) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
  RD_DISPATCH(dtype, launch_pdl(swiglu_kernel<T>, grid, SWIGLU_THREADS, 0, st, proj, (T*)out_t, F, m_total, cs));
  return cudaGetLastError();
}

// ---------------------------------------------------------------- the LLM's token per row (lowest index on ties)
// Philox-4x32-10 (Salmon et al., SC'11): counter (c0..c3), key (k0, k1) -> four words.
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
    const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
    c0 = h1 ^ c1 ^ k0; c1 = l1;
    c2 = h0 ^ c3 ^ k1; c3 = l0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}
// 32 random bits -> standard Gumbel noise: u = (top 23 bits + 1/2) / 2^23 lies in (0, 1) and is exact in fp32.
__device__ __forceinline__ float gumbel_of(uint32_t x) {
  const float u = ((float)(x >> 9) + 0.5f) * (1.0f / 8388608.0f);
  return -logf(-logf(u));
}

// SAMPLE = false: greedy token.  SAMPLE = true: a draw from softmax(logits / T) by the Gumbel-max rule (Section 3.4's
// rejection sampling for deterministic proposals: the LLM's own draw at a node, which acceptance compares with the
// node's children); the noise of vocabulary entry v depends on (seed; sequence, position of the token being chosen, v)
// only, so every row that predicts the same position of a sequence uses the same noise.
template <bool SAMPLE>
__global__ void __launch_bounds__(512) argmax_rows_kernel(float* __restrict__ logits, GemmOut proj, int V, int32_t* __restrict__ out,
                                   const int32_t* __restrict__ out_index, const int32_t* __restrict__ m_total, Sampling smp,
                                   const int32_t* __restrict__ row_seq, const int32_t* __restrict__ row_pos, int pos_add) {
  pdl_enter();
  __shared__ float sv[32];
  __shared__ int si[32];
  const int m = blockIdx.x;
  const int M = *m_total;
  if (m >= M) return;
  float* r = logits + (size_t)m * V;
  const GemmRows m_tiles = gemm_m_tiles(proj, M);
  uint32_t seq = 0, pos = 0;
  if (SAMPLE) {
    seq = row_seq ? (uint32_t)row_seq[m] : (uint32_t)m;
    pos = (uint32_t)(row_pos[m] + pos_add);
  }
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  // the complete logits are written back in place (later readers of the buffer see final values); four float4 per
  // thread and pass, every load of the four in flight before the first is used
  constexpr int ARG_BATCH = 4, ARG_FOLD = 2;
  for (int i0 = threadIdx.x * 4; i0 < V; i0 += blockDim.x * 4 * ARG_BATCH) {
    GemmPending4<ARG_FOLD> pd[ARG_BATCH];
#pragma unroll
    for (int u = 0; u < ARG_BATCH; ++u) {
      const int i = i0 + u * blockDim.x * 4;
      if (i < V) pd[u] = gemm_issue4<ARG_FOLD>(proj, m_tiles, m, i);
    }
#pragma unroll
    for (int u = 0; u < ARG_BATCH; ++u) {
      const int i = i0 + u * blockDim.x * 4;
      if (i < V) {
        const float4 q = gemm_finish4(proj, m_tiles, pd[u]);
        *reinterpret_cast<float4*>(r + i) = q;
        float e[4] = {q.x, q.y, q.z, q.w};
        if (SAMPLE) {
          const uint4 x = philox4x32_10((uint32_t)i >> 2, pos, seq, 0u, smp.k0, smp.k1);
          e[0] = e[0] * smp.inv_t + gumbel_of(x.x);
          e[1] = e[1] * smp.inv_t + gumbel_of(x.y);
          e[2] = e[2] * smp.inv_t + gumbel_of(x.z);
          e[3] = e[3] * smp.inv_t + gumbel_of(x.w);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (e[k] > bv || (e[k] == bv && i + k < bi)) { bv = e[k]; bi = i + k; }
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) { sv[w] = bv; si[w] = bi; }
  __syncthreads();
  if (w == 0) {
    const int nw = blockDim.x >> 5;
    bv = lane < nw ? sv[lane] : -INFINITY;
    bi = lane < nw ? si[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) out[out_index ? out_index[m] : m] = (bi == 0x7fffffff) ? 0 : bi;
  }
}

// logits: the projection's output buffer [M][V] (V a multiple of 4), completed in place.  With smp.inv_t > 0 row m
// draws the token at position row_pos[m] + pos_add of sequence row_seq[m] (row m itself where row_seq is null).
cudaError_t launch_argmax_rows(float* logits, const GemmOut& proj, int V, int32_t* out, const int32_t* out_index,
                               const int32_t* m_total, int m_max, const Sampling& smp, const int32_t* row_seq,
                               const int32_t* row_pos, int pos_add, cudaStream_t st) {
  if (smp.inv_t > 0.0f)
    launch_pdl(argmax_rows_kernel<true>, m_max, 512, 0, st, logits, proj, V, out, out_index, m_total, smp, row_seq, row_pos, pos_add);
  else
    launch_pdl(argmax_rows_kernel<false>, m_max, 512, 0, st, logits, proj, V, out, out_index, m_total, smp, row_seq, row_pos, pos_add);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- compact rows -> padded [B][NMAX] layout
__global__ void scatter_rows_kernel(const float* __restrict__ src, int width, float* __restrict__ dst,
                                    const int32_t* __restrict__ row_out_index, const int32_t* __restrict__ m_total) {
  pdl_enter();
  const int m = blockIdx.y;
  if (m >= *m_total) return;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < width) dst[(size_t)row_out_index[m] * width + i] = src[(size_t)m * width + i];
}

cudaError_t launch_scatter_rows(const float* src, int width, float* dst, const int32_t* row_out_index,
                                const int32_t* m_total, int m_max, cudaStream_t st) {
  dim3 grid((width + 255) / 256, m_max);
  launch_pdl(scatter_rows_kernel, grid, 256, 0, st, src, width, dst, row_out_index, m_total);
  return cudaGetLastError();
}

template <typename T>
__global__ void cast_rows_kernel(const float* __restrict__ src, T* __restrict__ dst, int n) {
  pdl_enter();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = from_f<T>(src[i]);
}

cudaError_t launch_cast_rows(int dtype, const float* src, void* dst, int n, cudaStream_t st) {
  RD_DISPATCH(dtype, launch_pdl(cast_rows_kernel<T>, (n + 255) / 256, 256, 0, st, src, (T*)dst, n));
  return cudaGetLastError();
}

__global__ void fill_i32_kernel(int32_t* p, int32_t v, int n) {
  pdl_enter();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

cudaError_t launch_fill_i32(int32_t* p, int32_t v, int n, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  launch_pdl(fill_i32_kernel, (n + 255) / 256, 256, 0, st, p, v, n);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- row tables
// Verification: the packed rows of all sequences are laid out back to back (compact), so the
// projections see M = sum_b n[b] rows.  Row (b, n): token = packed token, position = ctx_b + depth,
// provisional cache slot ctx_b + n, attends cache [0, ctx_b) plus its mask row.
__global__ void build_rows_tree_kernel(rd_packed pk, const int32_t* __restrict__ ctx, int32_t* row_tok, int32_t* row_seq,
                                       int32_t* row_pos, int32_t* row_slot, int32_t* row_ncache, int32_t* row_local,
                                       int32_t* row_out_index, int32_t* seq_off, int32_t* seq_order, int32_t* m_total, Dims dm,
                                       int B, int* status) {
  pdl_enter();
  extern __shared__ int32_t off[];  // [B+1]
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int b = 0; b < B; ++b) {
      off[b] = acc;
      int n = pk.n[b];
      if (n < 0 || n > dm.NMAX) { atomicOr(status, DEV_ERR_INDEX_RANGE); n = min(max(n, 0), dm.NMAX); }
      acc += n;
    }
    off[B] = acc;
    *m_total = acc;
  }
  __syncthreads();
  for (int b = threadIdx.x; b <= B; b += blockDim.x) seq_off[b] = off[b];
  // The sequences by key extent, longest first (ties by index): attention kernels whose CTAs walk a whole sequence's keys
  // hand the long sequences out first, so that the last CTAs to start are short ones.  Ranked by counting.
  if (seq_order)
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
      const int kb = ctx[b] + (off[b + 1] - off[b]);
      int rank = 0;
      for (int o = 0; o < B; ++o) {
        const int ko = ctx[o] + (off[o + 1] - off[o]);
        rank += (ko > kb || (ko == kb && o < b)) ? 1 : 0;
      }
      seq_order[rank] = b;
    }
  for (int idx = threadIdx.x; idx < B * dm.NMAX; idx += blockDim.x) {
    const int b = idx / dm.NMAX, n = idx - b * dm.NMAX;
    if (n >= off[b + 1] - off[b]) continue;
    const int m = off[b] + n;
    int t = pk.tokens[idx];
    if (t < 0 || t >= dm.V) { atomicOr(status, DEV_ERR_TOKEN_RANGE); t = min(max(t, 0), dm.V - 1); }
    row_tok[m] = t;
    row_seq[m] = b;
    row_pos[m] = pk.pos[idx];
    row_slot[m] = ctx[b] + n;
    row_ncache[m] = ctx[b];
    row_local[m] = n;
    row_out_index[m] = idx;
  }
}

cudaError_t launch_build_rows_tree(const rd_packed& pk, const int32_t* ctx, int32_t* row_tok, int32_t* row_seq,
                                   int32_t* row_pos, int32_t* row_slot, int32_t* row_ncache, int32_t* row_local,
                                   int32_t* row_out_index, int32_t* seq_off, int32_t* seq_order, int32_t* m_total,
                                   const Dims& dm, int B, int* status, cudaStream_t st) {
  launch_pdl(build_rows_tree_kernel, 1, 1024, (B + 1) * sizeof(int32_t), st, pk, ctx, row_tok, row_seq, row_pos, row_slot,
                                                                    row_ncache, row_local, row_out_index, seq_off,
                                                                    B <= 1024 ? seq_order : nullptr, m_total, dm, B, status);
  return cudaGetLastError();
}

// Autoregressive step: one row per sequence, the root token at position ctx_b.
__global__ void build_rows_ar_kernel(const int32_t* __restrict__ root, const int32_t* __restrict__ ctx, int32_t* row_tok,
                                     int32_t* row_seq, int32_t* row_pos, int32_t* row_slot, int32_t* row_ncache,
                                     int32_t* row_local, int32_t* row_out_index, int32_t* seq_off, int32_t* m_total,
                                     Dims dm, int B, int* status) {
  pdl_enter();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b == 0) { *m_total = B; seq_off[B] = B; }
  if (b >= B) return;
  seq_off[b] = b;
  int t = root[b];
  if (t < 0 || t >= dm.V) { atomicOr(status, DEV_ERR_TOKEN_RANGE); t = min(max(t, 0), dm.V - 1); }
  row_tok[b] = t;
  row_seq[b] = b;
  row_pos[b] = ctx[b];
  row_slot[b] = ctx[b];
  row_ncache[b] = ctx[b] + 1;
  row_local[b] = 0;
  row_out_index[b] = b;
}

cudaError_t launch_build_rows_ar(const int32_t* root, const int32_t* ctx, int32_t* row_tok, int32_t* row_seq,
                                 int32_t* row_pos, int32_t* row_slot, int32_t* row_ncache, int32_t* row_local,
                                 int32_t* row_out_index, int32_t* seq_off, int32_t* m_total, const Dims& dm, int B,
                                 int* status, cudaStream_t st) {
  launch_pdl(build_rows_ar_kernel, (B + 127) / 128, 128, 0, st, root, ctx, row_tok, row_seq, row_pos, row_slot, row_ncache,
                                                        row_local, row_out_index, seq_off, m_total, dm, B, status);
  return cudaGetLastError();
}

// After an AR forward: ctx += 1, root = greedy token, h = hidden of the row.
__global__ void ar_finish_kernel(const int32_t* __restrict__ argmax_c, const float* __restrict__ hidden_c, int32_t* ctx,
                                 int32_t* root, float* h, int32_t* token_out, int d) {
  pdl_enter();
  const int b = blockIdx.x;
  for (int i = threadIdx.x; i < d; i += blockDim.x) h[(size_t)b * d + i] = hidden_c[(size_t)b * d + i];
  if (threadIdx.x == 0) {
    ctx[b] += 1;
    root[b] = argmax_c[b];
    if (token_out) token_out[b] = argmax_c[b];
  }
}

cudaError_t launch_ar_finish(const int32_t* argmax_c, const float* hidden_c, int32_t* ctx, int32_t* root, float* h,
                             int32_t* token_out, const Dims& dm, int B, cudaStream_t st) {
  launch_pdl(ar_finish_kernel, B, 256, 0, st, argmax_c, hidden_c, ctx, root, h, token_out, dm.d);
  return cudaGetLastError();
}

// After a prefill pass: sequences whose last prompt token was in this pass take its hidden state.
__global__ void prefill_finish_kernel(const float* __restrict__ hidden_c, const int32_t* __restrict__ last_row, float* h,
                                      int d) {
  pdl_enter();
  const int b = blockIdx.x;
  const int r = last_row[b];
  if (r < 0) return;
  for (int i = threadIdx.x; i < d; i += blockDim.x) h[(size_t)b * d + i] = hidden_c[(size_t)r * d + i];
}

cudaError_t launch_prefill_finish(const float* hidden_c, const int32_t* last_row, float* h, int d, int B,
                                  cudaStream_t st) {
  launch_pdl(prefill_finish_kernel, B, 256, 0, st, hidden_c, last_row, h, d);
  return cudaGetLastError();
}

}  // namespace rd

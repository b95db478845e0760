// Small row-wise kernels of the verification forward (Section 3.4): embedding gather, RMSNorm,
// rotary embedding + KV-cache write, SwiGLU, row argmax, row tables.  All are bandwidth-trivial
// (activations of at most a few MB that stay in L2); they exist to feed the projections.
#include "rd_internal.cuh"

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
  RD_DISPATCH(dtype, embed_kernel<T><<<m_max, 256, 0, st>>>((const T*)emb, tok, x, d, V, m_total, status));
  return cudaGetLastError();
}

// ---------------------------------------------------------------- RMSNorm
// y = x / sqrt(mean(x^2) + eps) * gain, one block per row.
template <typename T>
__global__ void rmsnorm_kernel(const float* __restrict__ x, const T* __restrict__ gain, T* __restrict__ out_t,
                               float* __restrict__ out_f, int d, float eps, const int32_t* __restrict__ m_total) {
  __shared__ float sh[32];
  const int m = blockIdx.x;
  if (m >= *m_total) return;
  const float* xr = x + (size_t)m * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) { float v = xr[i]; ss += v * v; }
  ss = block_sum(ss, sh);
  const float r = rsqrtf(ss / (float)d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = xr[i] * r * to_f<T>(gain[i]);
    if (out_t) out_t[(size_t)m * d + i] = from_f<T>(v);
    if (out_f) out_f[(size_t)m * d + i] = v;
  }
}

cudaError_t launch_rmsnorm(int dtype, const float* x, const void* gain, void* out_t, float* out_f32, int d, float eps,
                           const int32_t* m_total, int m_max, cudaStream_t st) {
  RD_DISPATCH(dtype, rmsnorm_kernel<T><<<m_max, 256, 0, st>>>(x, (const T*)gain, (T*)out_t, out_f32, d, eps, m_total));
  return cudaGetLastError();
}

// ---------------------------------------------------------------- rotary embedding + KV write
// qkv: [M][3d] fp32 (Q | K | V).  Q is rotated in place; rotated K and V go to the cache slot of
// the row.  Pairing (i, i + hd/2), angle = pos * theta^(-2i/hd) (computed in double: positions
// reach several thousand and the angle's rounding error would otherwise scale with them).
template <typename T>
__global__ void rope_kv_kernel(float* __restrict__ qkv, T* __restrict__ kc, T* __restrict__ vc, RowTables rt, Dims dm,
                               int* status) {
  const int m = blockIdx.x;
  if (m >= *rt.m_total) return;
  const int b = rt.seq[m], slot = rt.slot[m], pos = rt.pos[m];
  const int d = dm.d, hd = dm.hd, half = hd >> 1;
  const bool slot_ok = slot >= 0 && slot < dm.max_ctx;
  if (!slot_ok && threadIdx.x == 0) atomicOr(status, DEV_ERR_CAPACITY);
  float* row = qkv + (size_t)m * 3 * d;
  const double l2t = log2((double)dm.theta);
  for (int idx = threadIdx.x; idx < dm.H * half; idx += blockDim.x) {
    const int h = idx / half, i = idx - h * half;
    const double ang = (double)pos * exp2(-(2.0 * i / hd) * l2t);
    double sd, cd;
    sincos(ang, &sd, &cd);
    const float c = (float)cd, s = (float)sd;
    const int o = h * hd + i;
    const float q1 = row[o], q2 = row[o + half];
    row[o] = q1 * c - q2 * s;
    row[o + half] = q2 * c + q1 * s;
    const float k1 = row[d + o], k2 = row[d + o + half];
    if (slot_ok) {
      const size_t base = (((size_t)b * dm.H + h) * dm.max_ctx + slot) * hd + i;
      kc[base] = from_f<T>(k1 * c - k2 * s);
      kc[base + half] = from_f<T>(k2 * c + k1 * s);
      vc[base] = from_f<T>(row[2 * d + o]);
      vc[base + half] = from_f<T>(row[2 * d + o + half]);
    }
  }
}

cudaError_t launch_rope_kv(int dtype, float* qkv, void* kcache, void* vcache, const RowTables& rt, const Dims& dm,
                           int m_max, int* status, cudaStream_t st) {
  RD_DISPATCH(dtype, rope_kv_kernel<T><<<m_max, 256, 0, st>>>(qkv, (T*)kcache, (T*)vcache, rt, dm, status));
  return cudaGetLastError();
}

// ---------------------------------------------------------------- SwiGLU
template <typename T>
__global__ void swiglu_kernel(const float* __restrict__ gu, T* __restrict__ out, int F, const int32_t* __restrict__ m_total) {
  const int m = blockIdx.y;
  if (m >= *m_total) return;
  const int f = blockIdx.x * blockDim.x + threadIdx.x;
  if (f >= F) return;
  const float g = gu[(size_t)m * 2 * F + f], u = gu[(size_t)m * 2 * F + F + f];
  out[(size_t)m * F + f] = from_f<T>(silu_f(g) * u);
}

cudaError_t launch_swiglu(int dtype, const float* gu, void* out_t, int F, const int32_t* m_total, int m_max,
                          cudaStream_t st) {
  dim3 grid((F + 255) / 256, m_max);
  RD_DISPATCH(dtype, swiglu_kernel<T><<<grid, 256, 0, st>>>(gu, (T*)out_t, F, m_total));
  return cudaGetLastError();
}

// ---------------------------------------------------------------- row argmax (lowest index on ties)
__global__ void argmax_rows_kernel(const float* __restrict__ logits, int V, int32_t* __restrict__ out,
                                   const int32_t* __restrict__ out_index, const int32_t* __restrict__ m_total) {
  __shared__ float sv[32];
  __shared__ int si[32];
  const int m = blockIdx.x;
  if (m >= *m_total) return;
  const float* r = logits + (size_t)m * V;
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  for (int i = threadIdx.x; i < V; i += blockDim.x) {
    const float v = r[i];
    if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
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

cudaError_t launch_argmax_rows(const float* logits, int V, int32_t* out, const int32_t* out_index,
                               const int32_t* m_total, int m_max, cudaStream_t st) {
  argmax_rows_kernel<<<m_max, 512, 0, st>>>(logits, V, out, out_index, m_total);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- compact rows -> padded [B][NMAX] layout
__global__ void scatter_rows_kernel(const float* __restrict__ src, int width, float* __restrict__ dst,
                                    const int32_t* __restrict__ row_out_index, const int32_t* __restrict__ m_total) {
  const int m = blockIdx.y;
  if (m >= *m_total) return;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < width) dst[(size_t)row_out_index[m] * width + i] = src[(size_t)m * width + i];
}

cudaError_t launch_scatter_rows(const float* src, int width, float* dst, const int32_t* row_out_index,
                                const int32_t* m_total, int m_max, cudaStream_t st) {
  dim3 grid((width + 255) / 256, m_max);
  scatter_rows_kernel<<<grid, 256, 0, st>>>(src, width, dst, row_out_index, m_total);
  return cudaGetLastError();
}

template <typename T>
__global__ void cast_rows_kernel(const float* __restrict__ src, T* __restrict__ dst, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = from_f<T>(src[i]);
}

cudaError_t launch_cast_rows(int dtype, const float* src, void* dst, int n, cudaStream_t st) {
  RD_DISPATCH(dtype, cast_rows_kernel<T><<<(n + 255) / 256, 256, 0, st>>>(src, (T*)dst, n));
  return cudaGetLastError();
}

__global__ void fill_i32_kernel(int32_t* p, int32_t v, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

cudaError_t launch_fill_i32(int32_t* p, int32_t v, int n, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  fill_i32_kernel<<<(n + 255) / 256, 256, 0, st>>>(p, v, n);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- row tables
// Verification: the packed rows of all sequences are laid out back to back (compact), so the
// projections see M = sum_b n[b] rows.  Row (b, n): token = packed token, position = ctx_b + depth,
// provisional cache slot ctx_b + n, attends cache [0, ctx_b) plus its mask row.
__global__ void build_rows_tree_kernel(rd_packed pk, const int32_t* __restrict__ ctx, int32_t* row_tok, int32_t* row_seq,
                                       int32_t* row_pos, int32_t* row_slot, int32_t* row_ncache, int32_t* row_local,
                                       int32_t* row_out_index, int32_t* m_total, Dims dm, int B, int* status) {
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
                                   int32_t* row_out_index, int32_t* m_total, const Dims& dm, int B, int* status,
                                   cudaStream_t st) {
  build_rows_tree_kernel<<<1, 1024, (B + 1) * sizeof(int32_t), st>>>(pk, ctx, row_tok, row_seq, row_pos, row_slot,
                                                                    row_ncache, row_local, row_out_index, m_total, dm,
                                                                    B, status);
  return cudaGetLastError();
}

// Autoregressive step: one row per sequence, the root token at position ctx_b.
__global__ void build_rows_ar_kernel(const int32_t* __restrict__ root, const int32_t* __restrict__ ctx, int32_t* row_tok,
                                     int32_t* row_seq, int32_t* row_pos, int32_t* row_slot, int32_t* row_ncache,
                                     int32_t* row_local, int32_t* row_out_index, int32_t* m_total, Dims dm, int B,
                                     int* status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b == 0) *m_total = B;
  if (b >= B) return;
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
                                 int32_t* row_out_index, int32_t* m_total, const Dims& dm, int B, int* status,
                                 cudaStream_t st) {
  build_rows_ar_kernel<<<(B + 127) / 128, 128, 0, st>>>(root, ctx, row_tok, row_seq, row_pos, row_slot, row_ncache,
                                                        row_local, row_out_index, m_total, dm, B, status);
  return cudaGetLastError();
}

// After an AR forward: ctx += 1, root = greedy token, h = hidden of the row.
__global__ void ar_finish_kernel(const int32_t* __restrict__ argmax_c, const float* __restrict__ hidden_c, int32_t* ctx,
                                 int32_t* root, float* h, int32_t* token_out, int d) {
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
  ar_finish_kernel<<<B, 256, 0, st>>>(argmax_c, hidden_c, ctx, root, h, token_out, dm.d);
  return cudaGetLastError();
}

// After a prefill pass: sequences whose last prompt token was in this pass take its hidden state.
__global__ void prefill_finish_kernel(const float* __restrict__ hidden_c, const int32_t* __restrict__ last_row, float* h,
                                      int d) {
  const int b = blockIdx.x;
  const int r = last_row[b];
  if (r < 0) return;
  for (int i = threadIdx.x; i < d; i += blockDim.x) h[(size_t)b * d + i] = hidden_c[(size_t)r * d + i];
}

cudaError_t launch_prefill_finish(const float* hidden_c, const int32_t* last_row, float* h, int d, int B,
                                  cudaStream_t st) {
  prefill_finish_kernel<<<B, 256, 0, st>>>(hidden_c, last_row, h, d);
  return cudaGetLastError();
}

}  // namespace rd

// Beam search over the RNN drafter (Sections 3.1, 3.2): the small kernels around the
// projections.  A drafter call t works on R = B*BW rows (call 1: B rows):
//   rnn:   s_t = SiLU([U W] [s_{t-1}; e_t] + b)        one projection over the concatenated input,
//                                                       finished by act_kernel
//   head:  x <- x + SiLU(A_l x + c_l), x_0 = [s_t, h]   one projection per layer, finished by act_kernel
//   out:   logits = O x                                  one projection
//   row_topk:   per row, log-sum-exp and the BW best logits (value desc, index asc)
//   beam_merge: per sequence, score_r + logit - lse_r over the BW*BW survivors, best BW in
//               (score desc, flat index r*V + v asc) order; reorders histories and states and
//               gathers the next call's input [s_t of the parent ; E[token]].
#include "rd_internal.cuh"
#include "gemm_out.cuh"
#include "pdl.cuh"

namespace rd {

#define RD_DISPATCH(dtype, ...)                                \
  if ((dtype) == RD_DTYPE_FP32) { using T = float; __VA_ARGS__; } \
  else { using T = __nv_bfloat16; __VA_ARGS__; }

// ---------------------------------------------------------------- call-1 input and s_1
// x[b] = [E[g_b], h_b] for the first call; the state half of se[r] = [s ; e] is E[g_b] = s_1 for
// every beam row r of b.
template <typename T>
__global__ void draft_init_kernel(const T* __restrict__ emb, const int32_t* __restrict__ root, const float* __restrict__ h,
                                  T* __restrict__ x_t, float* __restrict__ x_f, T* __restrict__ se_t, Dims dm,
                                  int* status) {
  pdl_enter();
  const int b = blockIdx.x;
  int g = root[b];
  if (g < 0 || g >= dm.V) {
    if (threadIdx.x == 0) atomicOr(status, DEV_ERR_TOKEN_RANGE);
    g = min(max(g, 0), dm.V - 1);
  }
  const int d = dm.d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const T e = emb[(size_t)g * d + i];
    x_t[(size_t)b * dm.dh + i] = e;
    x_f[(size_t)b * dm.dh + i] = to_f<T>(e);
    const float hv = h[(size_t)b * d + i];
    x_t[(size_t)b * dm.dh + dm.dr + i] = from_f<T>(hv);
    x_f[(size_t)b * dm.dh + dm.dr + i] = hv;
    for (int k = 0; k < dm.BW; ++k) se_t[((size_t)b * dm.BW + k) * (dm.dr + dm.d) + i] = e;
  }
}

cudaError_t launch_draft_init(int dtype, const void* emb, const int32_t* root, const float* h, void* x_t, float* x_f,
                              void* se_t, const Dims& dm, int B, int* status, cudaStream_t st) {
  RD_DISPATCH(dtype, launch_pdl(draft_init_kernel<T>, B, 256, 0, st, (const T*)emb, root, h, (T*)x_t, x_f, (T*)se_t, dm, status));
  return cudaGetLastError();
}

// h part of g_t = [s_t, h] for every beam row (constant over the calls of one step).
template <typename T>
__global__ void fill_h_kernel(const float* __restrict__ h, T* __restrict__ x_t, float* __restrict__ x_f, Dims dm) {
  pdl_enter();
  const int r = blockIdx.x, b = r / dm.BW;
  for (int i = threadIdx.x; i < dm.d; i += blockDim.x) {
    const float hv = h[(size_t)b * dm.d + i];
    x_t[(size_t)r * dm.dh + dm.dr + i] = from_f<T>(hv);
    x_f[(size_t)r * dm.dh + dm.dr + i] = hv;
  }
}

cudaError_t launch_fill_h(int dtype, const float* h, void* x_t, float* x_f, const Dims& dm, int B, cudaStream_t st) {
  RD_DISPATCH(dtype, launch_pdl(fill_h_kernel<T>, B * dm.BW, 256, 0, st, h, (T*)x_t, x_f, dm));
  return cudaGetLastError();
}

// ---------------------------------------------------------------- finish of a drafter projection
// out[m][n] = (resid ? resid[m][n] : 0) + SiLU(proj[m][n] + bias[n]), written as fp32 and in the
// storage type (the next projection's input).  Used for the RNN cell (no residual) and for the
// head's residual layers.
template <typename T>
__global__ void act_kernel(GemmOut proj, const T* __restrict__ bias, const float* __restrict__ resid, int ld_resid,
                           float* __restrict__ out_f, T* __restrict__ out_t, int ld_out, int N,
                           const int32_t* __restrict__ m_total) {
  pdl_enter();
  const int m = blockIdx.y;
  const int M = *m_total;
  if (m >= M) return;
  const int n = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (n >= N) return;
  const float4 q = gemm_value4(proj, gemm_m_tiles(proj, M), m, n);
  float v[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    v[k] = silu_f(v[k] + to_f<T>(bias[n + k]));
    if (resid) v[k] += resid[(size_t)m * ld_resid + n + k];
    out_f[(size_t)m * ld_out + n + k] = v[k];
    out_t[(size_t)m * ld_out + n + k] = from_f<T>(v[k]);
  }
}

cudaError_t launch_act(int dtype, const GemmOut& proj, const void* bias, const float* resid, int ld_resid, float* out_f,
                       void* out_t, int ld_out, int N, const int32_t* m_total, int m_max, cudaStream_t st) {
  dim3 grid((N / 4 + 255) / 256, m_max);
  RD_DISPATCH(dtype, launch_pdl(act_kernel<T>, grid, 256, 0, st, proj, (const T*)bias, resid, ld_resid, out_f, (T*)out_t,
                                ld_out, N, m_total));
  return cudaGetLastError();
}

// ---------------------------------------------------------------- per-row log-sum-exp + top-BW
// Ordering (value desc, index asc).  Selection is stateless: pass p picks the best element that
// comes strictly after the element picked by pass p-1, so nothing is marked or modified.
struct Cand {
  float v;
  int i;
};
__device__ __forceinline__ bool cand_before(float va, int ia, float vb, int ib) {  // a ranks before b
  return va > vb || (va == vb && ia < ib);
}
__device__ __forceinline__ Cand cand_best(Cand a, Cand b) { return cand_before(a.v, a.i, b.v, b.i) ? a : b; }
__device__ __forceinline__ Cand block_best(Cand c, Cand* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Cand t;
    t.v = __shfl_xor_sync(0xffffffffu, c.v, o);
    t.i = __shfl_xor_sync(0xffffffffu, c.i, o);
    c = cand_best(c, t);
  }
  __syncthreads();
  if (lane == 0) sh[w] = c;
  __syncthreads();
  Cand r = lane < nw ? sh[lane] : Cand{-INFINITY, 0x7fffffff};
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Cand t;
    t.v = __shfl_xor_sync(0xffffffffu, r.v, o);
    t.i = __shfl_xor_sync(0xffffffffu, r.i, o);
    r = cand_best(r, t);
  }
  return r;  // identical in every thread
}

// One CTA per row.  The row is read once into registers (TOPK_PER_THREAD values per thread); the BW
// selection passes then work on registers plus one block reduction each.
constexpr int TOPK_THREADS = 1024;
constexpr int TOPK_PER_THREAD = 32;  // V <= 32768

__global__ void __launch_bounds__(TOPK_THREADS) row_topk_kernel(GemmOut proj, int V, int BW, float* __restrict__ lse,
                                                                 float* __restrict__ val, int32_t* __restrict__ idx,
                                                                 const int32_t* __restrict__ m_total) {
  pdl_enter();
  __shared__ Cand sh[32];
  __shared__ float shf[32];
  const int r = blockIdx.x;
  const int m_tiles = gemm_m_tiles(proj, *m_total);
  // element (k, e) of this thread is column 4 * (threadIdx.x + (k / 4) * TOPK_THREADS) + k % 4
  float v[TOPK_PER_THREAD];
  Cand c{-INFINITY, 0x7fffffff};
#pragma unroll
  for (int k4 = 0; k4 < TOPK_PER_THREAD / 4; ++k4) {
    const int i = 4 * (threadIdx.x + k4 * TOPK_THREADS);
    float4 q = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    if (i < V) q = gemm_value4(proj, m_tiles, r, i);   // V is a multiple of 4
    v[4 * k4] = q.x; v[4 * k4 + 1] = q.y; v[4 * k4 + 2] = q.z; v[4 * k4 + 3] = q.w;
#pragma unroll
    for (int e = 0; e < 4; ++e) c = cand_best(c, Cand{v[4 * k4 + e], i < V ? i + e : 0x7fffffff});
  }
  const Cand top = block_best(c, sh);
  float s = 0.f;
#pragma unroll
  for (int k = 0; k < TOPK_PER_THREAD; ++k) s += expf(v[k] - top.v);  // exp(-inf) = 0 for the padding
  {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    __syncthreads();
    if (lane == 0) shf[w] = s;
    __syncthreads();
    s = lane < nw ? shf[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  }
  if (threadIdx.x == 0) {
    lse[r] = top.v + logf(s);
    val[(size_t)r * BW] = top.v;
    idx[(size_t)r * BW] = top.i;
  }
  Cand prev = top;
  for (int p = 1; p < BW; ++p) {
    Cand best{-INFINITY, 0x7fffffff};
#pragma unroll
    for (int k = 0; k < TOPK_PER_THREAD; ++k) {
      const int i = 4 * (threadIdx.x + (k >> 2) * TOPK_THREADS) + (k & 3);
      if (i < V && cand_before(prev.v, prev.i, v[k], i)) best = cand_best(best, Cand{v[k], i});
    }
    best = block_best(best, sh);
    if (threadIdx.x == 0) {
      val[(size_t)r * BW + p] = best.v;
      idx[(size_t)r * BW + p] = best.i == 0x7fffffff ? 0 : best.i;
    }
    prev = best;
  }
}

cudaError_t launch_row_topk(const GemmOut& proj, int V, int BW, float* lse, float* val, int32_t* idx, int rows,
                            const int32_t* m_total, cudaStream_t st) {
  if (V > TOPK_THREADS * TOPK_PER_THREAD) return cudaErrorInvalidValue;
  launch_pdl(row_topk_kernel, rows, TOPK_THREADS, 0, st, proj, V, BW, lse, val, idx, m_total);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- cross-row merge + reorder + gather
// call == 1: the single row's top-BW become the beams.  call >= 2: best BW of the BW*BW survivors.  Writes score_out[k], hist_out[k][0..call-1], and the next call's inputs
// se_t[k] = [s_t of the parent (read from s_new_f with row stride ld_s; skipped for call 1, where every
// beam keeps s_1) ; E[token_k]].  On the last call also the public outputs.
template <typename T>
__global__ void __launch_bounds__(256) beam_merge_kernel(int call, const float* __restrict__ lse,
                                                          const float* __restrict__ val, const int32_t* __restrict__ idx,
                                                          const float* __restrict__ score_in, float* __restrict__ score_out,
                                                          const int32_t* __restrict__ hist_in, int32_t* __restrict__ hist_out,
                                                          const T* __restrict__ emb, const float* __restrict__ s_new_f,
                                                          int ld_s, T* __restrict__ se_t, Dims dm,
                                                          int32_t* __restrict__ beams_out, float* __restrict__ scores_out) {
  pdl_enter();
  // grid = B * BW: every CTA of a sequence repeats the (tiny) selection over the BW*BW survivors and
  // then writes the outputs of ONE new beam, so the reorder/gather work is spread over BW CTAs.
  __shared__ Cand sh[32];
  __shared__ int sel_parent[128], sel_tok[128];
  __shared__ float sel_score[128];
  const int BW = dm.BW, L = dm.L, V = dm.V;
  const int b = blockIdx.x / BW, k = blockIdx.x - b * BW;
  const int rows = call == 1 ? 1 : BW;
  const int row0 = call == 1 ? b : b * BW;
  const int n_cand = rows * BW;
  Cand prev{INFINITY, -1};
  for (int p = 0; p <= k; ++p) {  // beams are ranked: beam k needs the first k+1 picks only
    Cand best{-INFINITY, 0x7fffffff};
    for (int c = threadIdx.x; c < n_cand; c += blockDim.x) {
      const int r = c / BW;
      const size_t o = (size_t)(row0 + r) * BW + (c - r * BW);
      const float base = call == 1 ? 0.f : score_in[row0 + r];
      const float sc = base + (val[o] - lse[row0 + r]);
      const int flat = r * V + idx[o];
      if (cand_before(prev.v, prev.i, sc, flat)) best = cand_best(best, Cand{sc, flat});
    }
    best = block_best(best, sh);
    if (threadIdx.x == 0) {
      sel_parent[p] = best.i / V;
      sel_tok[p] = best.i - (best.i / V) * V;
      sel_score[p] = best.v;
    }
    prev = best;
  }
  __syncthreads();
  const int orow = b * BW + k;
  const int prow = b * BW + sel_parent[k];
  const int tok = sel_tok[k];
  if (threadIdx.x == 0) {
    score_out[orow] = sel_score[k];
    for (int t = 0; t < call - 1; ++t) hist_out[(size_t)orow * L + t] = hist_in[(size_t)prow * L + t];
    hist_out[(size_t)orow * L + call - 1] = tok;
    if (call == L) {
      for (int t = 0; t < L - 1; ++t) beams_out[(size_t)orow * L + t] = hist_in[(size_t)prow * L + t];
      beams_out[(size_t)orow * L + L - 1] = tok;
      if (scores_out) scores_out[orow] = sel_score[k];
    }
  }
  if (call < L) {
    // gathers with 128-bit accesses (rows are 16-byte aligned: d is a multiple of 8)
    // next call's input row [s of the parent ; E[token]]
    constexpr int EV = 16 / sizeof(T);
    T* se = se_t + (size_t)orow * (dm.dr + dm.d);
    const uint4* e = reinterpret_cast<const uint4*>(emb + (size_t)tok * dm.d);
    uint4* eo = reinterpret_cast<uint4*>(se + dm.dr);
    for (int i = threadIdx.x; i < dm.d / EV; i += blockDim.x) eo[i] = e[i];
    if (call > 1) {
      const float4* s = reinterpret_cast<const float4*>(s_new_f + (size_t)prow * ld_s);
      T* so = se;
      for (int i = threadIdx.x; i < dm.dr / 4; i += blockDim.x) {
        const float4 v = s[i];
        so[4 * i] = from_f<T>(v.x); so[4 * i + 1] = from_f<T>(v.y); so[4 * i + 2] = from_f<T>(v.z); so[4 * i + 3] = from_f<T>(v.w);
      }
    }
  }
}

cudaError_t launch_beam_merge(int dtype, int call, const float* lse, const float* val, const int32_t* idx,
                              const float* score_in, float* score_out, const int32_t* hist_in, int32_t* hist_out,
                              const void* emb, const float* s_new_f, int ld_s, void* se_t, const Dims& dm, int B,
                              int32_t* beams_out, float* scores_out, cudaStream_t st) {
  RD_DISPATCH(dtype, launch_pdl(beam_merge_kernel<T>, B * dm.BW, 256, 0, st, call, lse, val, idx, score_in, score_out, hist_in, hist_out,
                                                           (const T*)emb, s_new_f, ld_s, (T*)se_t, dm,
                                                           beams_out, scores_out));
  return cudaGetLastError();
}

}  // namespace rd

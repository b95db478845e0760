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
constexpr int ACT_THREADS = 128;
constexpr int ACT_FOLD = 5;   // partial slots loaded up front (a 128-k-block tile cut over 28-unit ranges has up to 5 extra)

__device__ __forceinline__ void act_store4(float* p, float a, float b, float c, float d) { *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d); }
__device__ __forceinline__ void act_store4(__nv_bfloat16* p, float a, float b, float c, float d) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 u;
  u.x = *reinterpret_cast<const uint32_t*>(&lo);
  u.y = *reinterpret_cast<const uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = u;
}
template <typename T> __device__ __forceinline__ float4 act_bias4(const T* p);
template <> __device__ __forceinline__ float4 act_bias4<float>(const float* p) { return *reinterpret_cast<const float4*>(p); }
template <> __device__ __forceinline__ float4 act_bias4<__nv_bfloat16>(const __nv_bfloat16* p) {
  const uint2 g = *reinterpret_cast<const uint2*>(p);
  const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&g.x));
  const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&g.y));
  return make_float4(a.x, a.y, b.x, b.y);
}

// One float4 of one row per thread, small CTAs spread over all SMs (what bounds the kernel is the rate at
// which one SM pulls data out of the L2).  The bias is a weight and every address is a launch constant: both
// are dealt with before the wait; after it the thread loads, adds and stores.
template <typename T>
__global__ void __maxnreg__(88) act_kernel(GemmOut proj, const T* __restrict__ bias, const float* resid, int ld_resid,
                                           float* __restrict__ out_f, T* __restrict__ out_t, int ld_out, int N,
                                           const int32_t* __restrict__ m_total, ChainSync cs) {
  chain_begin(cs);
  const int m = blockIdx.y;
  const int n = (blockIdx.x * ACT_THREADS + threadIdx.x) * 4;
  const bool active = n < N;
  const bool fast = proj.m_tiles_max == 1 && (proj.partial == nullptr || proj.all_work);
  const size_t stride = gemm_slot_stride(proj);
  GemmSrc src;
  float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
  const float* rp = resid ? resid + (size_t)m * ld_resid + n : nullptr;
  float* of = out_f + (size_t)m * ld_out + n;
  T* ot = out_t + (size_t)m * ld_out + n;
  if (active) {
    bv = act_bias4<T>(bias + n);
    if (fast) { src = gemm_src(proj, 1, m, n); gemm_src_pin(src); }
    asm volatile("" : "+l"(rp), "+l"(of), "+l"(ot));
  }
  // inside a chain the row count, written ahead of the chain, is requested before the wait
  const bool early = cs.signal_ptr != nullptr && cs.wait_ptr != nullptr;
  int M = early ? *m_total : 0;
  chain_wait_cta(cs);
  if (!early) M = *m_total;
  if (m < M && active) {
    float4 q;
    float4 rv = make_float4(0.f, 0.f, 0.f, 0.f);
    if (fast) {
      const auto dat = gemm_load4<ACT_FOLD>(src, stride);
      if (rp) rv = __ldcg(reinterpret_cast<const float4*>(rp));
      q = gemm_sum4(src, stride, dat);
    } else {
      if (rp) rv = __ldcg(reinterpret_cast<const float4*>(rp));
      q = gemm_value4(proj, gemm_m_tiles(proj, M), m, n);
    }
    const float y0 = rv.x + silu_f(q.x + bv.x), y1 = rv.y + silu_f(q.y + bv.y), y2 = rv.z + silu_f(q.z + bv.z),
                y3 = rv.w + silu_f(q.w + bv.w);
    act_store4(of, y0, y1, y2, y3);
    act_store4(ot, y0, y1, y2, y3);
  }
  chain_exit(cs);
}

// N, ld_resid, ld_out multiples of 4 (8 for bf16 outputs); bias 16-byte aligned.
cudaError_t launch_act(int dtype, const GemmOut& proj, const void* bias, const float* resid, int ld_resid, float* out_f,
                       void* out_t, int ld_out, int N, const int32_t* m_total, int m_max, Chain* chain, cudaStream_t st) {
  dim3 grid((N / 4 + ACT_THREADS - 1) / ACT_THREADS, m_max);
  const ChainSync cs = chain ? chain->link(grid.x * grid.y, true) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
  RD_DISPATCH(dtype, launch_pdl(act_kernel<T>, grid, ACT_THREADS, 0, st, proj, (const T*)bias, resid, ld_resid, out_f,
                                (T*)out_t, ld_out, N, m_total, cs));
  return cudaGetLastError();
}

// ---------------------------------------------------------------- selection: log-softmax, top-BW, beam pruning
// Ordering of candidates: (value desc, index asc).  Selection is stateless: round p picks the best
// element that comes strictly after the one picked by round p-1, so nothing is marked or modified.
struct Cand {
  float v;
  int i;
};
__device__ __forceinline__ bool cand_before(float va, int ia, float vb, int ib) {  // a ranks before b
  return va > vb || (va == vb && ia < ib);
}
__device__ __forceinline__ Cand cand_best(Cand a, Cand b) { return cand_before(a.v, a.i, b.v, b.i) ? a : b; }
__device__ __forceinline__ Cand warp_best(Cand c) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Cand t;
    t.v = __shfl_xor_sync(0xffffffffu, c.v, o);
    t.i = __shfl_xor_sync(0xffffffffu, c.i, o);
    c = cand_best(c, t);
  }
  return c;  // identical in every lane
}
__device__ __forceinline__ float block_reduce_sum(float s, float* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  __syncthreads();
  if (lane == 0) sh[w] = s;
  __syncthreads();
  s = lane < nw ? sh[lane] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  return s;
}

constexpr int SEL_THREADS = 1024;
constexpr int SEL_MAX_BW = 128;
constexpr int SEL_LIST_CAP = 1024;  // elements at or above the selection threshold

// One CTA per drafter row r (a live beam, or the single row of call 1).
//  1. the row's logits (projection output + partial slots) into registers, 32 per thread;
//  2. log-sum-exp of the row; a threshold that at least BW values reach (the BW-th largest per-thread
//     maximum, found with warp shuffles); the few values at or above it go to a shared list that warp 0
//     ranks.  Each value is touched a constant number of times, whatever BW is;
//  3. the last CTA of a sequence to finish (atomic counter, no waiting) prunes the BW x BW survivors
//     score_r + logit - lse_r to the BW best in (score desc, flat index r*V + v asc) order, writes the
//     new scores and histories, and gathers the next call's input rows [s_t of the parent ; E[token]].
template <typename T>
__global__ void __launch_bounds__(SEL_THREADS) draft_select_kernel(
    GemmOut proj, int call, float* __restrict__ lse, float* __restrict__ val, int32_t* __restrict__ idx,
    const float* __restrict__ score_in, float* __restrict__ score_out, const int32_t* __restrict__ hist_in,
    int32_t* __restrict__ hist_out, const T* __restrict__ emb, const float* __restrict__ s_new_f, int ld_s,
    T* __restrict__ se_t, Dims dm, int32_t* __restrict__ beams_out, float* __restrict__ scores_out,
    int32_t* __restrict__ counters, const int32_t* __restrict__ m_total, unsigned long long* dbg, ChainSync cs) {
  unsigned long long t_dbg[8];
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[0]));
  chain_enter(cs);
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[1]));
  extern __shared__ __align__(16) uint8_t sel_smem[];
  Cand* wl = reinterpret_cast<Cand*>(sel_smem);            // [32 warps][BW] per-warp survivors; reused by the pruning
  __shared__ float shf[32];
  __shared__ Cand sh_top[SEL_MAX_BW];
  __shared__ int sel_parent[SEL_MAX_BW], sel_tok[SEL_MAX_BW];
  __shared__ float sel_score[SEL_MAX_BW];
  __shared__ int s_last, s_count;
  __shared__ float s_tau;
  const int BW = dm.BW, L = dm.L, V = dm.V;
  const int r = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const GemmRows m_tiles = gemm_m_tiles(proj, *m_total);
  Cand* cl = wl + 32 * BW;   // [SEL_LIST_CAP] values at or above the threshold
  // ---- 1. logits into shared memory (compact loops from here on: the kernel runs once per launch,
  // so straight-line code would be bound by instruction fetch)
  float* zrow = reinterpret_cast<float*>(cl + SEL_LIST_CAP);   // [V]
  float tmax = -INFINITY;
#pragma unroll 4
  for (int i = 4 * threadIdx.x; i < V; i += 4 * SEL_THREADS) {
    const float4 q = gemm_value4<2>(proj, m_tiles, r, i);   // V is a multiple of 4
    *reinterpret_cast<float4*>(zrow + i) = q;
    tmax = fmaxf(tmax, fmaxf(fmaxf(q.x, q.y), fmaxf(q.z, q.w)));
  }
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[2]));
  // ---- 2a. a threshold that at least BW elements reach: the BW-th largest of the 1024 per-thread maxima
  // (per warp BW rounds over one value per lane, then warp 0 over the 32 x BW survivors)
  {
    Cand prev{INFINITY, -1};
    for (int p = 0; p < BW; ++p) {
      Cand best{-INFINITY, 0x7fffffff};
      if (cand_before(prev.v, prev.i, tmax, lane)) best = Cand{tmax, lane};
      best = warp_best(best);
      if (lane == 0) wl[warp * BW + p] = best;   // index unused below
      prev = best;
    }
  }
  // ---- 2b. log-sum-exp of the row
  float wmax = tmax;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) wmax = fmaxf(wmax, __shfl_xor_sync(0xffffffffu, wmax, o));
  __syncthreads();
  if (lane == 0) shf[warp] = wmax;
  if (threadIdx.x == 0) s_count = 0;
  __syncthreads();
  float rmax = shf[lane];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, o));
  float s = 0.f;
#pragma unroll 4
  for (int i = 4 * threadIdx.x; i < V; i += 4 * SEL_THREADS) {
    const float4 q = *reinterpret_cast<const float4*>(zrow + i);
    s += __expf(q.x - rmax) + __expf(q.y - rmax) + __expf(q.z - rmax) + __expf(q.w - rmax);
  }
  s = block_reduce_sum(s, shf);   // also orders the wl writes before warp 0 reads them
  const float row_lse = rmax + logf(s);
  if (warp == 0) {
    Cand pv{INFINITY, -1};
    for (int p = 0; p < BW; ++p) {
      Cand best{-INFINITY, 0x7fffffff};
      for (int c = lane; c < 32 * BW; c += 32) {
        const float x = wl[c].v;
        if (cand_before(pv.v, pv.i, x, c)) best = cand_best(best, Cand{x, c});
      }
      best = warp_best(best);
      pv = best;
    }
    if (lane == 0) s_tau = pv.v;   // -inf when the row has fewer than BW values
  }
  __syncthreads();
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[3]));
  // ---- 2c. every element that reaches the threshold goes to a short list; warp 0 ranks the list
  const float tau = s_tau;
#pragma unroll 4
  for (int i = 4 * threadIdx.x; i < V; i += 4 * SEL_THREADS) {
    const float4 q = *reinterpret_cast<const float4*>(zrow + i);
    const float e[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (e[k] >= tau) {
        const int slot = atomicAdd(&s_count, 1);
        if (slot < SEL_LIST_CAP) cl[slot] = Cand{e[k], i + k};
      }
    }
  }
  __syncthreads();
  const int n_list = s_count;
  if (n_list <= SEL_LIST_CAP) {
    if (warp == 0) {
      Cand pv{INFINITY, -1};
      for (int p = 0; p < BW; ++p) {
        Cand best{-INFINITY, 0x7fffffff};
        for (int c = lane; c < n_list; c += 32) {
          const Cand x = cl[c];
          if (cand_before(pv.v, pv.i, x.v, x.i)) best = cand_best(best, x);
        }
        best = warp_best(best);
        if (lane == 0) {
          val[(size_t)r * BW + p] = best.v;
          idx[(size_t)r * BW + p] = best.i == 0x7fffffff ? 0 : best.i;
        }
        pv = best;
      }
    }
  } else {
    // more ties at the threshold than the list holds: rank by rounds over all values (slow, exact)
    Cand prev{INFINITY, -1};
    for (int p = 0; p < BW; ++p) {
      Cand best{-INFINITY, 0x7fffffff};
      for (int i = threadIdx.x; i < V; i += SEL_THREADS)
        if (cand_before(prev.v, prev.i, zrow[i], i)) best = cand_best(best, Cand{zrow[i], i});
      best = warp_best(best);
      __syncthreads();
      if (lane == 0) wl[warp] = best;
      __syncthreads();
      best = warp_best(wl[lane]);
      if (threadIdx.x == 0) {
        val[(size_t)r * BW + p] = best.v;
        idx[(size_t)r * BW + p] = best.i == 0x7fffffff ? 0 : best.i;
      }
      prev = best;
    }
  }
  if (threadIdx.x == 0) lse[r] = row_lse;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[4]));
  // ---- 3. pruning by the sequence's last CTA
  const int rows = call == 1 ? 1 : BW;
  const int b = call == 1 ? r : r / BW;
  const int row0 = call == 1 ? b : b * BW;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int old = atomicAdd(counters + b, 1);
    s_last = (old == rows - 1) ? 1 : 0;
    if (old == rows - 1) counters[b] = 0;
  }
  __syncthreads();
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[5]));
  if (!s_last) {
    chain_exit(cs);
    return;
  }
  __threadfence();
  const int n_cand = rows * BW;
  // candidates into shared memory: score and flat index
  for (int c = threadIdx.x; c < n_cand; c += blockDim.x) {
    const int rr = c / BW;
    const size_t o = (size_t)(row0 + rr) * BW + (c - rr * BW);
    const float base = call == 1 ? 0.f : score_in[row0 + rr];
    wl[c] = Cand{base + (__ldcg(val + o) - __ldcg(lse + row0 + rr)), rr * V + __ldcg(idx + o)};
  }
  __syncthreads();
  if (warp == 0) {
    Cand pv{INFINITY, -1};
    for (int p = 0; p < BW; ++p) {
      Cand best{-INFINITY, 0x7fffffff};
      for (int c = lane; c < n_cand; c += 32) {
        const Cand x = wl[c];
        if (cand_before(pv.v, pv.i, x.v, x.i)) best = cand_best(best, x);
      }
      best = warp_best(best);
      if (lane == 0) sh_top[p] = best;
      pv = best;
    }
  }
  __syncthreads();
  for (int k = threadIdx.x; k < BW; k += blockDim.x) {
    const Cand c = sh_top[k];
    const int parent = c.i / V, tok = c.i - parent * V;
    sel_parent[k] = parent; sel_tok[k] = tok; sel_score[k] = c.v;
    const int orow = b * BW + k, prow = b * BW + parent;
    score_out[orow] = c.v;
    for (int t = 0; t < call - 1; ++t) hist_out[(size_t)orow * L + t] = hist_in[(size_t)prow * L + t];
    hist_out[(size_t)orow * L + call - 1] = tok;
    if (call == L) {
      for (int t = 0; t < L - 1; ++t) beams_out[(size_t)orow * L + t] = hist_in[(size_t)prow * L + t];
      beams_out[(size_t)orow * L + L - 1] = tok;
      if (scores_out) scores_out[orow] = c.v;
    }
  }
  __syncthreads();
  if (call < L) {
    // next call's input rows [s of the parent ; E[token]], 128-bit accesses (d, d_rnn multiples of 8)
    constexpr int EV = 16 / sizeof(T);
    const int ev = dm.d / EV, sv = dm.dr / 4;
    for (int item = threadIdx.x; item < BW * ev; item += blockDim.x) {
      const int k = item / ev, i = item - k * ev;
      const uint4* e = reinterpret_cast<const uint4*>(emb + (size_t)sel_tok[k] * dm.d);
      reinterpret_cast<uint4*>(se_t + (size_t)(b * BW + k) * (dm.dr + dm.d) + dm.dr)[i] = e[i];
    }
    if (call > 1) {
      for (int item = threadIdx.x; item < BW * sv; item += blockDim.x) {
        const int k = item / sv, i = item - k * sv;
        const float4 q = reinterpret_cast<const float4*>(s_new_f + (size_t)(b * BW + sel_parent[k]) * ld_s)[i];
        T* so = se_t + (size_t)(b * BW + k) * (dm.dr + dm.d) + 4 * i;
        so[0] = from_f<T>(q.x); so[1] = from_f<T>(q.y); so[2] = from_f<T>(q.z); so[3] = from_f<T>(q.w);
      }
    }
  }
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[6]));
  if (dbg && threadIdx.x == 0) {
    for (int i = 0; i < 7; ++i) dbg[i] = t_dbg[i];
  }
  chain_exit(cs);
}

// ---------------------------------------------------------------- selection in two short kernels (BW <= 64)
// The one-CTA-per-row kernel above pulls a whole row of logits through one SM and ranks it there; with a
// handful of rows that leaves most of the GPU idle for tens of microseconds.  Here every row is cut into S
// segments (rows x S CTAs, about one per SM): a segment's CTA folds its logits, and reduces them to the
// segment's maximum, its sum of exponentials and its BW best candidates.  A second kernel with one CTA per
// surviving beam merges the segments of its sequence's rows (log-sum-exp, BW best per row), prunes the
// BW x BW candidates in (score desc, flat index asc) order up to its own rank, and writes that beam's score,
// history and next input row.  Both orders are the ones of the single-kernel path.
// (value desc, index asc) as the unsigned order of one 64-bit key; 0 is below every candidate.
__device__ __forceinline__ unsigned long long cand_key(float v, int i) {
  uint32_t u = __float_as_uint(v);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)i);
}
__device__ __forceinline__ float key_value(unsigned long long k) {
  if (k == 0ull) return -INFINITY;
  const uint32_t u = (uint32_t)(k >> 32);
  return __uint_as_float((u & 0x80000000u) ? (u ^ 0x80000000u) : ~u);
}
__device__ __forceinline__ int key_index(unsigned long long k) {
  return k == 0ull ? 0x7fffffff : (int)(0xFFFFFFFFu - (uint32_t)(k & 0xFFFFFFFFull));
}
__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long k) {
  const uint32_t hi = (uint32_t)(k >> 32), lo = (uint32_t)k;
  const uint32_t mh = __reduce_max_sync(0xffffffffu, hi);
  const uint32_t ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
  return ((unsigned long long)mh << 32) | ml;
}

constexpr int SEG_THREADS = 256;
constexpr int SEG_ITEMS_MAX = 4;     // float4 per thread at most (the kernel is instantiated for 1, 2 and 4)
constexpr int SEG_FOLD = 2;
constexpr int SEG_MAX_CAND = 512;    // S * BW candidates per row at most
constexpr int SEG_LIST_CAP = 1024;   // candidates at or above a segment's threshold that the counting path takes
constexpr int MRG_THREADS = 256;
constexpr int MRG_MAX_BW = 64;       // the merge kernel ranks BW x BW keys in shared memory
constexpr int MRG_NARROW_BW = 16;    // up to here the narrow variant (candidates re-read from shared memory) is the faster

template <int SEG_ITEMS>
__global__ void __maxnreg__(88) draft_seg_kernel(GemmOut proj, int V, int BW, int seg_len4, float* __restrict__ seg_max,
                                                 float* __restrict__ seg_sum, float* __restrict__ seg_val,
                                                 int32_t* __restrict__ seg_idx, const int32_t* __restrict__ m_total,
                                                 ChainSync cs) {
  chain_begin(cs);
  __shared__ float shf[32];
  const int r = blockIdx.y, sgm = blockIdx.x, S = gridDim.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool fast = proj.m_tiles_max == 1 && (proj.partial == nullptr || proj.all_work);
  const size_t stride = gemm_slot_stride(proj);
  GemmSrc src[SEG_ITEMS];
  int col[SEG_ITEMS];
  bool ok[SEG_ITEMS];
#pragma unroll
  for (int k = 0; k < SEG_ITEMS; ++k) {
    const int j = threadIdx.x + k * SEG_THREADS;
    col[k] = 4 * (sgm * seg_len4 + j);
    ok[k] = j < seg_len4 && col[k] < V;
    if (fast && ok[k]) { src[k] = gemm_src(proj, 1, r, col[k]); gemm_src_pin(src[k]); }
  }
  chain_wait_cta(cs);
  float v[SEG_ITEMS][4];
  if (fast) {
    GemmData4<SEG_FOLD> dat[SEG_ITEMS];
#pragma unroll
    for (int k = 0; k < SEG_ITEMS; ++k)
      if (ok[k]) dat[k] = gemm_load4<SEG_FOLD>(src[k], stride);
#pragma unroll
    for (int k = 0; k < SEG_ITEMS; ++k) {
      float4 q = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      if (ok[k]) q = gemm_sum4(src[k], stride, dat[k]);
      v[k][0] = q.x; v[k][1] = q.y; v[k][2] = q.z; v[k][3] = q.w;
    }
  } else {
    const GemmRows m_tiles = gemm_m_tiles(proj, *m_total);
#pragma unroll
    for (int k = 0; k < SEG_ITEMS; ++k) {
      float4 q = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      if (ok[k]) q = gemm_value4<SEG_FOLD>(proj, m_tiles, r, col[k]);
      v[k][0] = q.x; v[k][1] = q.y; v[k][2] = q.z; v[k][3] = q.w;
    }
  }
  // ---- segment maximum and sum of exponentials
  float tmax = -INFINITY;
#pragma unroll
  for (int k = 0; k < SEG_ITEMS; ++k)
#pragma unroll
    for (int e = 0; e < 4; ++e) tmax = fmaxf(tmax, v[k][e]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
  if (lane == 0) shf[warp] = tmax;
  __syncthreads();
  float smax = lane < SEG_THREADS / 32 ? shf[lane] : -INFINITY;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, o));
  float sum = 0.f;
  if (smax > -INFINITY) {
#pragma unroll
    for (int k = 0; k < SEG_ITEMS; ++k)
#pragma unroll
      for (int e = 0; e < 4; ++e) sum += __expf(v[k][e] - smax);   // exp(-inf) = 0 for the padding
  }
  sum = block_reduce_sum(sum, shf);
  if (threadIdx.x == 0) { seg_max[(size_t)r * S + sgm] = smax; seg_sum[(size_t)r * S + sgm] = sum; }
  // ---- the segment's BW best in (value desc, index asc) order.  Every candidate becomes one 64-bit key whose
  // unsigned order is that order (ordered value bits, then the complemented index): keys are unique.
  unsigned long long key[SEG_ITEMS * 4];
#pragma unroll
  for (int k = 0; k < SEG_ITEMS; ++k)
#pragma unroll
    for (int e = 0; e < 4; ++e) key[k * 4 + e] = ok[k] ? cand_key(v[k][e], col[k] + e) : 0ull;
  constexpr int NK = SEG_ITEMS * 4;
  // A threshold that at least BW candidates reach -- the BW-th largest of the threads' own maxima, ranked by counting --,
  // then the candidates at or above it go to a shared list that is ranked by counting as well.  Every key is touched
  // a constant number of times, whatever BW is (BW rounds of a block-wide maximum took 54 us per call at beam
  // width 64).  Exactly BW threads hold a maximum at or above the threshold, each with at most NK keys: the list
  // holds BW * NK keys at most.
  static_assert(MRG_MAX_BW * SEG_ITEMS_MAX * 4 <= SEG_LIST_CAP, "the list takes every key of BW threads");
  __shared__ unsigned long long s_tmax[SEG_THREADS];
  __shared__ unsigned long long s_list[SEG_LIST_CAP];
  __shared__ unsigned long long s_tau;
  __shared__ int s_n;
  unsigned long long tk = 0ull;
#pragma unroll
  for (int q = 0; q < NK; ++q) tk = max(tk, key[q]);
  s_tmax[threadIdx.x] = tk;
  if (threadIdx.x == 0) { s_n = 0; s_tau = 0ull; }
  __syncthreads();
  if (tk != 0ull) {
    int rank = 0;
#pragma unroll 8
    for (int j = 0; j < SEG_THREADS; ++j) rank += s_tmax[j] > tk ? 1 : 0;
    if (rank == BW - 1) s_tau = tk;   // keys are unique: one thread at most
  }
  __syncthreads();
  const unsigned long long tau = s_tau;   // 0: fewer than BW threads hold a candidate, every candidate qualifies
#pragma unroll
  for (int q = 0; q < NK; ++q)
    if (key[q] != 0ull && key[q] >= tau) {
      const int pos = atomicAdd(&s_n, 1);
      if (pos < SEG_LIST_CAP) s_list[pos] = key[q];
    }
  __syncthreads();
  const int n = min(s_n, SEG_LIST_CAP);
  float* out_v = seg_val + ((size_t)r * S + sgm) * BW;
  int32_t* out_i = seg_idx + ((size_t)r * S + sgm) * BW;
  for (int i = threadIdx.x; i < n; i += SEG_THREADS) {
    const unsigned long long k = s_list[i];
    int rank = 0;
    for (int j = 0; j < n; ++j) rank += s_list[j] > k ? 1 : 0;
    if (rank < BW) { out_v[rank] = key_value(k); out_i[rank] = key_index(k); }
  }
  for (int p = n + threadIdx.x; p < BW; p += SEG_THREADS) { out_v[p] = key_value(0ull); out_i[p] = key_index(0ull); }
  chain_exit(cs);
}

// Second of the three selection kernels: one CTA per drafter row.  The row's S segments each bring their maximum,
// their sum of exponentials and their BW best candidates; the CTA forms the row's log-sum-exp and ranks the S * BW
// candidates by counting (every key is unique: the index is part of it), so the BW best leave in order with one pass
// over shared memory per candidate instead of BW rounds of a maximum search.  Output: top[r][p], p < BW, the keys
// (cumulative score, flat index row-in-sequence * V + token) of the row's BW best continuations, best first; 0 where a
// row has fewer candidates.  Without this kernel every one of a sequence's BW merging CTAs repeated this work for all
// BW rows (178 us per call at beam width 64).
constexpr int ROWTOP_THREADS = 256;
static_assert(SEG_MAX_CAND <= 2 * ROWTOP_THREADS, "two candidates per thread");
__global__ void __launch_bounds__(ROWTOP_THREADS) draft_rowtop_kernel(int S, int call, int BW, int V, const float* __restrict__ seg_max,
                                                                      const float* __restrict__ seg_sum, const float* __restrict__ seg_val,
                                                                      const int32_t* __restrict__ seg_idx, const float* __restrict__ score_in,
                                                                      unsigned long long* __restrict__ top, ChainSync cs) {
  chain_enter(cs);
  __shared__ unsigned long long keys[SEG_MAX_CAND];
  __shared__ unsigned long long out[MRG_MAX_BW];
  __shared__ float s_lse;
  const int r = blockIdx.x;
  const int rr = call == 1 ? 0 : r % BW;     // the row's index inside its sequence (call 1: one row per sequence)
  const int n = S * BW;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int c = threadIdx.x; c < n; c += ROWTOP_THREADS) {
    const float cv = __ldcg(seg_val + (size_t)r * n + c);
    const int ci = __ldcg(seg_idx + (size_t)r * n + c);
    keys[c] = ci == 0x7fffffff ? 0ull : cand_key(cv, ci);
  }
  if (threadIdx.x < BW) out[threadIdx.x] = 0ull;
  if (warp == 0) {
    // log-sum-exp of the row from its segments (S <= 32: one per lane)
    const float sm = lane < S ? __ldcg(seg_max + (size_t)r * S + lane) : -INFINITY;
    const float ss = lane < S ? __ldcg(seg_sum + (size_t)r * S + lane) : 0.f;
    float m = sm;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float sum = sm > -INFINITY ? ss * __expf(sm - m) : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) s_lse = m + logf(sum);
  }
  __syncthreads();
  const float base = call == 1 ? 0.f : __ldcg(score_in + r);
  const float row_lse = s_lse;
  // a thread ranks its two candidates (c and c + 256; SEG_MAX_CAND = 2 * ROWTOP_THREADS) in one pass: every key read
  // from shared memory (a broadcast) serves both comparisons, eight reads in flight at a time
  {
    const int c0 = threadIdx.x, c1 = threadIdx.x + ROWTOP_THREADS;
    const unsigned long long k0 = c0 < n ? keys[c0] : 0ull, k1 = c1 < n ? keys[c1] : 0ull;
    int r0 = 0, r1 = 0;
#pragma unroll 8
    for (int j = 0; j < n; ++j) {
      const unsigned long long x = keys[j];
      r0 += x > k0 ? 1 : 0;
      r1 += x > k1 ? 1 : 0;
    }
    if (k0 != 0ull && r0 < BW) out[r0] = cand_key(base + (key_value(k0) - row_lse), rr * V + key_index(k0));
    if (k1 != 0ull && r1 < BW) out[r1] = cand_key(base + (key_value(k1) - row_lse), rr * V + key_index(k1));
  }
  __syncthreads();
  if (threadIdx.x < BW) top[(size_t)r * BW + threadIdx.x] = out[threadIdx.x];
  chain_exit(cs);
}

template <typename T, bool WIDE>
__global__ void __launch_bounds__(MRG_THREADS) draft_merge_kernel(
    int call, const unsigned long long* __restrict__ top_g, float* __restrict__ score_out,
    const int32_t* __restrict__ hist_in, int32_t* __restrict__ hist_out, const T* __restrict__ emb,
    const float* __restrict__ s_new_f, int ld_s, T* __restrict__ se_t, Dims dm, int32_t* __restrict__ beams_out,
    float* __restrict__ scores_out, unsigned long long* dbg, ChainSync cs) {
  unsigned long long t_dbg[4] = {0, 0, 0, 0};
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[0]));
  chain_enter(cs);
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[1]));
  extern __shared__ unsigned long long top[];   // rows * BW keys (dynamic: 32 KB at beam width 64)
  __shared__ Cand s_win;
  const int BW = dm.BW, L = dm.L, V = dm.V;
  const int kout = blockIdx.x, b = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int rows = call == 1 ? 1 : BW;
  const int row0 = call == 1 ? b : b * BW;
  // the rows' BW best continuations each (draft_rowtop_kernel), in row order
  for (int c = threadIdx.x; c < rows * BW; c += MRG_THREADS) top[c] = __ldcg(top_g + (size_t)row0 * BW + c);
  if constexpr (WIDE) {
    __shared__ unsigned long long s_tmax[MRG_THREADS];
    __shared__ unsigned long long s_list[SEG_LIST_CAP];
    __shared__ unsigned long long s_tau;
    __shared__ int s_n;
    __syncthreads();
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[2]));
    // The beam of rank kout among the rows * BW candidates, (score desc, flat index asc), in a constant number of
    // steps: every thread holds its share of the candidates in registers; the (kout + 1)-th largest of the threads'
    // own maxima (ranked by counting) is a threshold that at least kout + 1 candidates reach; the candidates at or
    // above it -- those of exactly kout + 1 threads, KPT each at most -- go to a list that is ranked by counting.
    // (kout + 1 rounds of a block-wide maximum took 28 us per call at beam width 64.)
    {
      const int n_cand = rows * BW;
      constexpr int KPT = MRG_MAX_BW * MRG_MAX_BW / MRG_THREADS;
      static_assert(MRG_MAX_BW * KPT <= SEG_LIST_CAP, "the list takes every key of kout + 1 threads");
      unsigned long long key[KPT];
      unsigned long long tk = 0ull;
  #pragma unroll
      for (int j = 0; j < KPT; ++j) {
        const int c = threadIdx.x + MRG_THREADS * j;
        key[j] = c < n_cand ? top[c] : 0ull;
        tk = max(tk, key[j]);
      }
      s_tmax[threadIdx.x] = tk;
      if (threadIdx.x == 0) { s_n = 0; s_tau = 0ull; s_win = Cand{-INFINITY, 0}; }
      __syncthreads();
      if (tk != 0ull) {
        int rank = 0;
  #pragma unroll 8
        for (int j = 0; j < MRG_THREADS; ++j) rank += s_tmax[j] > tk ? 1 : 0;
        if (rank == kout) s_tau = tk;   // keys are unique: one thread at most
      }
      __syncthreads();
      const unsigned long long tau = s_tau;   // 0: at most kout threads hold a candidate, every candidate qualifies
  #pragma unroll
      for (int j = 0; j < KPT; ++j)
        if (key[j] != 0ull && key[j] >= tau) {
          const int pos = atomicAdd(&s_n, 1);
          if (pos < SEG_LIST_CAP) s_list[pos] = key[j];
        }
      __syncthreads();
      const int n = min(s_n, SEG_LIST_CAP);
      for (int i = threadIdx.x; i < n; i += MRG_THREADS) {
        const unsigned long long k = s_list[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += s_list[j] > k ? 1 : 0;
        if (rank == kout) s_win = Cand{key_value(k), key_index(k)};   // (fewer candidates than beams cannot happen: BW <= V)
      }
    }
  } else {
    // narrow beams: the final ranking has a few candidates per lane of one warp
    __syncthreads();
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[2]));
    // the beam of rank kout among the rows * BW candidates, (score desc, flat index asc)
    if (warp == 0) {
      const int n_cand = rows * BW;
      unsigned long long pv = ~0ull;
      for (int p = 0; p <= kout; ++p) {
        unsigned long long mine = 0ull;
        for (int c = lane; c < n_cand; c += 32) {
          const unsigned long long x = top[c];
          mine = max(mine, x < pv ? x : 0ull);
        }
        pv = warp_max_key(mine);
      }
      if (lane == 0) s_win = Cand{key_value(pv), pv == 0ull ? 0 : key_index(pv)};   // (fewer candidates than beams cannot happen: BW <= V)
    }
  }
  __syncthreads();
  const Cand win = s_win;
  const int parent = win.i / V, tok = win.i - parent * V;
  const int orow = b * BW + kout, prow = b * BW + parent;
  if (threadIdx.x == 0) {
    score_out[orow] = win.v;
    for (int t = 0; t < call - 1; ++t) hist_out[(size_t)orow * L + t] = __ldcg(hist_in + (size_t)prow * L + t);
    hist_out[(size_t)orow * L + call - 1] = tok;
    if (call == L) {
      for (int t = 0; t < L - 1; ++t) beams_out[(size_t)orow * L + t] = __ldcg(hist_in + (size_t)prow * L + t);
      beams_out[(size_t)orow * L + L - 1] = tok;
      if (scores_out) scores_out[orow] = win.v;
    }
  }
  if (call < L) {
    // this beam's input row of the next call: [s of the parent ; E[token]], 128-bit accesses
    constexpr int EV = 16 / sizeof(T);
    const int ev = dm.d / EV, sv = dm.dr / 4;
    const uint4* e = reinterpret_cast<const uint4*>(emb + (size_t)tok * dm.d);
    uint4* eo = reinterpret_cast<uint4*>(se_t + (size_t)orow * (dm.dr + dm.d) + dm.dr);
    for (int i = threadIdx.x; i < ev; i += MRG_THREADS) eo[i] = e[i];
    if (call > 1) {
      const float4* sp = reinterpret_cast<const float4*>(s_new_f + (size_t)prow * ld_s);
      T* so = se_t + (size_t)orow * (dm.dr + dm.d);
      for (int i = threadIdx.x; i < sv; i += MRG_THREADS) {
        const float4 q = __ldcg(sp + i);
        act_store4(so + 4 * i, q.x, q.y, q.z, q.w);
      }
    }
  }
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[3]));
  if (dbg && threadIdx.x == 0) {
    atomicMin(dbg + 0, t_dbg[0]); atomicMin(dbg + 1, t_dbg[1]); atomicMax(dbg + 2, t_dbg[2]); atomicMax(dbg + 6, t_dbg[3]);
  }
  chain_exit(cs);
}

// Segments per row for the two-kernel selection, or 0 when the shape does not fit it.
int draft_select_segments(const Dims& dm, int rows, int grid_hint) {
  if (dm.BW > MRG_MAX_BW || (dm.V & 3)) return 0;
  int S = grid_hint / (rows > 0 ? rows : 1);
  const int s_cap = SEG_MAX_CAND / dm.BW < 32 ? SEG_MAX_CAND / dm.BW : 32;
  if (S > s_cap) S = s_cap;
  const int v4 = dm.V / 4;
  const int s_min = (v4 + SEG_THREADS * SEG_ITEMS_MAX - 1) / (SEG_THREADS * SEG_ITEMS_MAX);
  if (S < s_min) S = s_min;
  if (S < 1) S = 1;
  if (S > s_cap) return 0;
  return S;
}

// Once per handle (and so per device): opt-in of the one-kernel selection's shared-memory row (opted in by init).
cudaError_t drafter_prepare(int dtype) {
  const int top_bytes = MRG_MAX_BW * MRG_MAX_BW * (int)sizeof(unsigned long long);
  cudaError_t e = dtype == RD_DTYPE_FP32
                      ? cudaFuncSetAttribute(draft_merge_kernel<float, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, top_bytes)
                      : cudaFuncSetAttribute(draft_merge_kernel<__nv_bfloat16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, top_bytes);
  if (e != cudaSuccess) return e;
  return dtype == RD_DTYPE_FP32
             ? cudaFuncSetAttribute(draft_select_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)
             : cudaFuncSetAttribute(draft_select_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

// rows = B (call 1) or B * BW.  counters: [B] zero between launches.
cudaError_t launch_draft_select(int dtype, const GemmOut& proj, int call, float* lse, float* val, int32_t* idx,
                                const float* score_in, float* score_out, const int32_t* hist_in, int32_t* hist_out,
                                const void* emb, const float* s_new_f, int ld_s, void* se_t, const Dims& dm, int B,
                                int32_t* beams_out, float* scores_out, int32_t* counters, const int32_t* m_total,
                                unsigned long long* dbg, const SelectScratch& sc, Chain* chain, cudaStream_t st) {
  if (dm.BW > SEL_MAX_BW) return cudaErrorInvalidValue;
  const int rows = call == 1 ? B : B * dm.BW;
  const int S = sc.seg_max ? draft_select_segments(dm, rows, sc.grid_hint) : 0;
  if (S > 0) {
    const int seg_len4 = (dm.V / 4 + S - 1) / S;
    dim3 g1(S, rows);
    const ChainSync c1 = chain ? chain->link(g1.x * g1.y, true) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
    const int items = (seg_len4 + SEG_THREADS - 1) / SEG_THREADS;
#define RD_SEG_LAUNCH(ITEMS)                                                                                             \
  launch_pdl(draft_seg_kernel<ITEMS>, g1, SEG_THREADS, 0, st, proj, dm.V, dm.BW, seg_len4, sc.seg_max, sc.seg_sum,         \
             sc.seg_val, sc.seg_idx, m_total, c1)
    if (items <= 1) RD_SEG_LAUNCH(1);
    else if (items == 2) RD_SEG_LAUNCH(2);
    else RD_SEG_LAUNCH(4);
#undef RD_SEG_LAUNCH
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // the rows' BW best continuations, one CTA per row
    const ChainSync c15 = chain ? chain->link((unsigned)rows, true) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
    launch_pdl(draft_rowtop_kernel, rows, ROWTOP_THREADS, 0, st, S, call, dm.BW, dm.V, (const float*)sc.seg_max, (const float*)sc.seg_sum,
               (const float*)sc.seg_val, (const int32_t*)sc.seg_idx, score_in, sc.top, c15);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    dim3 g2(dm.BW, B);
    const ChainSync c2 = chain ? chain->link(g2.x * g2.y) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
    const size_t top_bytes = (size_t)(call == 1 ? 1 : dm.BW) * dm.BW * sizeof(unsigned long long);
    if (dm.BW > MRG_NARROW_BW) {
      constexpr bool WIDE_ = true;
      RD_DISPATCH(dtype, launch_pdl(draft_merge_kernel<T, WIDE_>, g2, MRG_THREADS, top_bytes, st, call, (const unsigned long long*)sc.top,
                                    score_out, hist_in, hist_out, (const T*)emb, s_new_f, ld_s, (T*)se_t, dm, beams_out,
                                    scores_out, dbg, c2));
    } else {
      constexpr bool WIDE_ = false;
      RD_DISPATCH(dtype, launch_pdl(draft_merge_kernel<T, WIDE_>, g2, MRG_THREADS, top_bytes, st, call, (const unsigned long long*)sc.top,
                                    score_out, hist_in, hist_out, (const T*)emb, s_new_f, ld_s, (T*)se_t, dm, beams_out,
                                    scores_out, dbg, c2));
    }
    return cudaGetLastError();
  }
  const size_t select = ((size_t)32 * dm.BW + SEL_LIST_CAP) * sizeof(Cand) + (size_t)dm.V * sizeof(float);
  const size_t prune = (size_t)dm.BW * dm.BW * sizeof(Cand);
  const size_t smem = select > prune ? select : prune;
  if (smem > 200 * 1024) return cudaErrorInvalidValue;   // vocabulary too large for the shared-memory row
  const ChainSync cs = chain ? chain->link((unsigned)rows) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
  RD_DISPATCH(dtype, launch_pdl(draft_select_kernel<T>, rows, SEL_THREADS, smem, st, proj, call, lse, val, idx, score_in,
                                score_out, hist_in, hist_out, (const T*)emb, s_new_f, ld_s, (T*)se_t, dm, beams_out,
                                scores_out, counters, m_total, dbg, cs));
  return cudaGetLastError();
}

}  // namespace rd

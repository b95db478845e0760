// Dynamic tree attention packing (Section 3.3, Appendix A.1) and greedy acceptance with KV-cache
// compaction (Section 3.4).  Integer work on at most a few thousand entries per sequence: one CTA
// per sequence, everything staged in shared memory, no host involvement.
#include <mutex>

#include "rd_internal.cuh"
#include "pdl.cuh"

namespace rd {

// ---------------------------------------------------------------- pack
// beam' = [root | beam] is [BW][C], C = L+1.  Thread (i, j):
//   owner(i,j) = the first candidate k <= i with beam'[k][0..j] == beam'[i][0..j]   (dedup_prefix)
//   keep(i,j)  = owner == i; packed index = exclusive scan of keep in row-major order (pack_beam)
//   unpack[i][j] = packed index of (owner, j); pos = ctx + j; parent = unpack[i][j-1];
//   mask row = bits unpack[i][0..j].
constexpr int PACK_MAX_ENTRIES = 1024;

__global__ void __launch_bounds__(1024) pack_kernel(const int32_t* __restrict__ beams, const int32_t* __restrict__ root,
                                                     const int32_t* __restrict__ ctx, rd_packed out, Dims dm, int no_tree) {
  pdl_enter();
  __shared__ int32_t tok[PACK_MAX_ENTRIES];
  __shared__ int32_t owner[PACK_MAX_ENTRIES];
  __shared__ int32_t scan[PACK_MAX_ENTRIES];
  __shared__ int32_t warp_tot[32];
  const int b = blockIdx.x, BW = dm.BW, L = dm.L, C = L + 1, E = BW * C;
  const int t = threadIdx.x;
  const int i = t / C, j = t - i * C;
  if (t < E) tok[t] = (j == 0) ? root[b] : beams[((size_t)b * BW + i) * L + (j - 1)];
  __syncthreads();
  int keep = 0, own = 0;
  if (t < E) {
    if (no_tree) {
      own = (j == 0) ? 0 : i;
    } else {
      own = i;
      for (int k = 0; k < i; ++k) {
        bool same = true;
        for (int c = 1; c <= j; ++c) same = same && (tok[k * C + c] == tok[i * C + c]);  // column 0 is the shared root
        if (same) { own = k; break; }
      }
    }
    keep = (own == i);
    owner[t] = own;
  }
  // exclusive scan of keep over t (row-major order)
  const int lane = t & 31, w = t >> 5;
  int incl = keep;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_tot[w] = incl;
  __syncthreads();
  if (w == 0) {
    int v = warp_tot[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += u;
    }
    warp_tot[lane] = v;  // inclusive totals
  }
  __syncthreads();
  const int excl = incl - keep + (w > 0 ? warp_tot[w - 1] : 0);
  if (t < E) scan[t] = excl;
  const int N = warp_tot[31];
  __syncthreads();

  const size_t rb = (size_t)b * dm.NMAX;
  // padding rows first (disjoint from kept rows)
  for (int n = N + t; n < dm.NMAX; n += blockDim.x) {
    out.tokens[rb + n] = 0;
    out.pos[rb + n] = 0;
    out.parent[rb + n] = -1;
    for (int wd = 0; wd < dm.MW; ++wd) out.mask[(rb + n) * dm.MW + wd] = 0u;
  }
  if (t == 0) out.n[b] = N;
  if (t < E) {
    const int u = scan[owner[t] * C + j];
    out.unpack[((size_t)b * BW + i) * C + j] = u;
    if (keep) {
      out.tokens[rb + excl] = tok[t];
      out.pos[rb + excl] = ctx[b] + j;
      out.parent[rb + excl] = (j == 0) ? -1 : scan[owner[i * C + j - 1] * C + j - 1];
      uint32_t* mr = out.mask + (rb + excl) * dm.MW;
      for (int wd = 0; wd < dm.MW; ++wd) mr[wd] = 0u;
      for (int c = 0; c <= j; ++c) {
        const int a = scan[owner[i * C + c] * C + c];
        mr[a >> 5] |= 1u << (a & 31);
      }
    }
  }
}

cudaError_t launch_pack(const int32_t* beams, const int32_t* root, const int32_t* ctx, const rd_packed& out,
                        const Dims& dm, int B, int no_tree, cudaStream_t st) {
  launch_pdl(pack_kernel, B, 1024, 0, st, beams, root, ctx, out, dm, no_tree);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- accept
// a_i = longest j with beam[i][j'] == llm_argmax[unpack[i][j']] for all j' < j; a = max_i a_i, best = the
// lowest such i; bonus = llm_argmax[unpack[best][a]]; next h = hidden[unpack[best][a]].
// Saves the old context length for the compaction kernel and advances ctx by 1 + a.
__global__ void __launch_bounds__(256) accept_kernel(const int32_t* __restrict__ beams, rd_packed pk,
                                                      const int32_t* __restrict__ argmax, const float* __restrict__ hidden,
                                                      int32_t* ctx, int32_t* root, float* h, rd_accept_out out,
                                                      int32_t* n_accept_ws, int32_t* best_ws, int32_t* ctx_prev, Dims dm,
                                                      int* status) {
  pdl_enter();
  __shared__ int sh_a[8], sh_i[8];
  __shared__ int s_a, s_best, s_node;
  const int b = blockIdx.x, BW = dm.BW, L = dm.L, C = L + 1;
  const size_t rb = (size_t)b * dm.NMAX;
  int a = -1, bi = 0x7fffffff;
  for (int i = threadIdx.x; i < BW; i += blockDim.x) {
    int ai = 0;
    while (ai < L) {
      const int node = pk.unpack[((size_t)b * BW + i) * C + ai];
      if (node < 0 || node >= dm.NMAX) { atomicOr(status, DEV_ERR_INDEX_RANGE); break; }
      if (beams[((size_t)b * BW + i) * L + ai] != argmax[rb + node]) break;
      ++ai;
    }
    if (ai > a || (ai == a && i < bi)) { a = ai; bi = i; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const int oa = __shfl_xor_sync(0xffffffffu, a, o), oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (oa > a || (oa == a && oi < bi)) { a = oa; bi = oi; }
  }
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) { sh_a[w] = a; sh_i[w] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int k = 1; k < (int)(blockDim.x >> 5); ++k)
      if (sh_a[k] > a || (sh_a[k] == a && sh_i[k] < bi)) { a = sh_a[k]; bi = sh_i[k]; }
    int node = pk.unpack[((size_t)b * BW + bi) * C + a];
    if (node < 0 || node >= dm.NMAX) { atomicOr(status, DEV_ERR_INDEX_RANGE); node = 0; }
    s_a = a; s_best = bi; s_node = node;
    const int bonus = argmax[rb + node];
    if (out.n_accept) out.n_accept[b] = a;
    if (out.best) out.best[b] = bi;
    if (out.tokens) {
      for (int j = 0; j < C; ++j)
        out.tokens[(size_t)b * C + j] = j < a ? beams[((size_t)b * BW + bi) * L + j] : (j == a ? bonus : -1);
    }
    n_accept_ws[b] = a;
    best_ws[b] = bi;
    ctx_prev[b] = ctx[b];
    ctx[b] += 1 + a;
    root[b] = bonus;
  }
  __syncthreads();
  const float* src = hidden + (rb + s_node) * dm.d;
  for (int i = threadIdx.x; i < dm.d; i += blockDim.x) h[(size_t)b * dm.d + i] = src[i];
}

// Compaction: the accepted path's K/V rows move from provisional slots ctx + unpack[best][j] to
// ctx + j, j = 1..a.  Sources are strictly increasing and never below their destination, so the
// moves are done in order of j; one CTA per (sequence, layer x {K,V}) handles all heads.
template <typename T>
__global__ void __launch_bounds__(256) compact_kv_kernel(T* __restrict__ kv, rd_packed pk,
                                                          const int32_t* __restrict__ n_accept,
                                                          const int32_t* __restrict__ best,
                                                          const int32_t* __restrict__ ctx_prev, Dims dm, int* status) {
  pdl_enter();
  const int b = blockIdx.x, plane = blockIdx.y;  // plane = layer*2 + {0:K, 1:V}
  const int a = n_accept[b];
  if (a <= 0) return;
  const int c0 = ctx_prev[b], C = dm.L + 1;
  T* base = kv + ((size_t)plane * dm.B + b) * dm.H * (size_t)dm.max_ctx * dm.hd;
  const int per_row = dm.H * dm.hd;  // elements moved per path node in this plane
  for (int j = 1; j <= a; ++j) {
    const int node = pk.unpack[((size_t)b * dm.BW + best[b]) * C + j];
    const int src = c0 + node, dst = c0 + j;
    if (node < j || src >= dm.max_ctx) {
      if (threadIdx.x == 0) atomicOr(status, DEV_ERR_INDEX_RANGE);
      return;
    }
    if (src != dst) {
      for (int e = threadIdx.x; e < per_row; e += blockDim.x) {
        const int hh = e / dm.hd, x = e - hh * dm.hd;
        T* head = base + (size_t)hh * dm.max_ctx * dm.hd;
        head[(size_t)dst * dm.hd + x] = head[(size_t)src * dm.hd + x];
      }
    }
    __syncthreads();
  }
}

cudaError_t launch_accept(int dtype, const int32_t* beams, const rd_packed& pk, const int32_t* argmax,
                          const float* hidden, void* kcache, int32_t* ctx, int32_t* root, float* h,
                          const rd_accept_out& out, int32_t* n_accept_ws, int32_t* best_ws, int32_t* ctx_prev,
                          const Dims& dm, int B, int* status, cudaStream_t st) {
  launch_pdl(accept_kernel, B, 256, 0, st, beams, pk, argmax, hidden, ctx, root, h, out, n_accept_ws, best_ws, ctx_prev, dm,
                                   status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 grid(B, dm.n_layers * 2);
  if (dtype == RD_DTYPE_FP32)
    launch_pdl(compact_kv_kernel<float>, grid, 256, 0, st, (float*)kcache, pk, n_accept_ws, best_ws, ctx_prev, dm, status);
  else
    launch_pdl(compact_kv_kernel<__nv_bfloat16>, grid, 256, 0, st, (__nv_bfloat16*)kcache, pk, n_accept_ws, best_ws, ctx_prev,
                                                           dm, status);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- scratch that needs no allocation
// The accept and compaction kernels hand three small per-sequence values to each other (accepted
// length, best candidate, previous context length).  redrafter_accept keeps them in the caller's
// workspace; redrafter_accept_static keeps them here, in memory that is part of the loaded library,
// for callers that cannot allocate.  Every GPU that loads the library holds these 48 KB until exit.
constexpr int ACCEPT_STATIC_MAX_BATCH = 4096;
static __device__ __align__(256) int32_t g_accept_scratch[3 * ACCEPT_STATIC_MAX_BATCH];

int accept_static_max_batch() { return ACCEPT_STATIC_MAX_BATCH; }

// Device address of the static scratch on the CURRENT device.  In host code the array's name is only a
// handle for the runtime, not an address a kernel can use, so the address is asked for once per device
// and remembered.
cudaError_t accept_static_scratch(int32_t** n_accept, int32_t** best, int32_t** ctx_prev) {
  constexpr int MAX_DEVICES = 64;
  static int32_t* base[MAX_DEVICES] = {};
  static std::mutex mu;   // host threads may make their first call on a device at the same time
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (base[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_accept_scratch);
    if (e != cudaSuccess) return e;
    base[dev] = static_cast<int32_t*>(p);
  }
  *n_accept = base[dev];
  *best = base[dev] + ACCEPT_STATIC_MAX_BATCH;
  *ctx_prev = base[dev] + 2 * ACCEPT_STATIC_MAX_BATCH;
  return cudaSuccess;
}

}  // namespace rd

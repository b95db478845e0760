// Where a projection's result lives until its consumer folds it.
//
// The tensor-core projection is a stream-K kernel: CTA c owns the contiguous unit range
// [c*U/G, (c+1)*U/G) of the (row tile, weight tile or tile pair, k-block) list, so a tile's k-range
// may be cut among several CTAs.  The kernel applies no epilogue and does no cross-CTA reduction.  The contributor that
// holds a tile's first k-block writes its sum to the fp32 output `raw`; every other contributor
// (its range then starts inside that tile, so it has exactly one such segment) writes its sum to
// its own slot of `partial`.  The kernel that consumes the projection (norm, rotary, SwiGLU,
// argmax, ...) adds the slots to `raw` in CTA order -- a fixed order, so results are
// deterministic -- while it does its own work.  This keeps fences, atomics and the serial
// reduction out of the weight-streaming kernel.
#pragma once
#include <stdint.h>

namespace rd {

struct GemmOut {
  const float* raw;      // [M][ld]
  const float* partial;  // [grid][mt * 128 (x 2 in pair mode)], nullptr when nothing is cut (CUDA-core path)
  int ld;
  int nkb, n_tiles, mt, grid, m_tiles_max;   // mt: most rows of a row tile; m_tiles_max: most row tiles of the launch
  int all_work;          // every CTA has a non-empty range for any row count (units >= CTAs)
  int pair;              // 1: a unit is (pair of adjacent tiles, k-block); a slot holds two tiles, even one first
  int small32;           // (units + 1) * CTAs stays below 2^31 for any row count of the launch: 32-bit index arithmetic
};

// Floats per partial slot (one slot per CTA).
__host__ __device__ __forceinline__ size_t gemm_slot_stride(const GemmOut& g) { return (size_t)g.mt * 128 * (g.pair ? 2 : 1); }

// Unit range of CTA c: [c*U/G, (c+1)*U/G).
__host__ __device__ __forceinline__ long long gemm_range_begin(long long c, long long U, long long G) { return c * U / G; }
// The CTA whose range holds unit u (the largest c with range_begin(c) <= u).
__host__ __device__ __forceinline__ int gemm_cta_of_unit(long long u, long long U, long long G) {
  const long long c = ((u + 1) * G - 1) / U;
  return (int)(c > G - 1 ? G - 1 : c);
}

// Row tiles of a launch over M rows: their number and the rows of each.  A launch laid out for several row tiles of
// at most g.mt rows uses the fewest tiles that hold M rows and makes them equal (a multiple of 16 rows), so that no
// tile is mostly padding.
struct GemmRows {
  int n, rows;
  __host__ __device__ GemmRows(int n_ = 1, int rows_ = 0) : n(n_), rows(rows_) {}
};
__host__ __device__ __forceinline__ GemmRows gemm_row_tiles(int mt, int m_tiles_max, int M) {
  if (m_tiles_max == 1) return GemmRows(1, mt);
  int n = (M + mt - 1) / mt;
  if (n < 1) n = 1;
  int rows = ((M + n - 1) / n + 15) & ~15;
  if (rows < 16) rows = 16;
  if (rows > mt) rows = mt;
  return GemmRows(n, rows);
}
__device__ __forceinline__ GemmRows gemm_m_tiles(const GemmOut& g, int M) { return gemm_row_tiles(g.mt, g.m_tiles_max, M); }

// Contributors of the tile that holds (m, n) other than the first: CTAs c_first+1 .. c_last.
struct GemmFold {
  int c_next, c_last;   // first non-first contributor, last contributor
  size_t off;           // element offset of (m, n) inside a slot
};
__device__ __forceinline__ GemmFold gemm_fold(const GemmOut& g, GemmRows m_tiles, int m, int n) {
  const int n_tile = n >> 7, row = n & 127;
  GemmFold f;
  if (m_tiles.n == 1) {
    // one row tile (the decode-time case): 32-bit arithmetic, (units + 1) * CTAs stays far below 2^31
    // (in pair mode the units run over pairs of tiles, and the odd tile sits in the second half of a slot)
    const uint32_t group = g.pair ? (uint32_t)(n_tile >> 1) : (uint32_t)n_tile;
    const uint32_t n_groups = g.pair ? (uint32_t)((g.n_tiles + 1) >> 1) : (uint32_t)g.n_tiles;
    const uint32_t U = n_groups * g.nkb, G = g.grid, tu0 = group * g.nkb;
    const uint32_t cf = ((tu0 + 1) * G - 1) / U, cl = ((tu0 + g.nkb) * G - 1) / U;
    f.c_next = (int)(cf > G - 1 ? G - 1 : cf) + 1;
    f.c_last = (int)(cl > G - 1 ? G - 1 : cl);
    f.off = (size_t)m * 128 + row + ((g.pair && (n_tile & 1)) ? (size_t)g.mt * 128 : 0);
    return f;
  }
  // several row tiles: units run over (row tile, tile or pair of tiles, k-block)
  const int m_tile = m / m_tiles.rows, col = m - m_tile * m_tiles.rows;
  const int group = g.pair ? (n_tile >> 1) : n_tile, n_groups = g.pair ? ((g.n_tiles + 1) >> 1) : g.n_tiles;
  f.off = (size_t)col * 128 + row + ((g.pair && (n_tile & 1)) ? (size_t)g.mt * 128 : 0);
  if (g.small32) {   // the usual case; 64-bit divisions cost the consuming kernels more than their loads
    const uint32_t U = (uint32_t)n_groups * m_tiles.n * g.nkb, G = g.grid, tu0 = ((uint32_t)m_tile * n_groups + group) * g.nkb;
    const uint32_t cf = ((tu0 + 1) * G - 1) / U, cl = ((tu0 + g.nkb) * G - 1) / U;
    f.c_next = (int)(cf > G - 1 ? G - 1 : cf) + 1;
    f.c_last = (int)(cl > G - 1 ? G - 1 : cl);
    return f;
  }
  const long long t = (long long)m_tile * n_groups + group;
  const long long U = (long long)n_groups * m_tiles.n * g.nkb, G = g.grid;
  const long long tu0 = t * g.nkb;
  f.c_next = gemm_cta_of_unit(tu0, U, G) + 1;
  f.c_last = gemm_cta_of_unit(tu0 + g.nkb - 1, U, G);
  return f;
}
// True when CTA c has work (with fewer units than CTAs some ranges are empty).
__device__ __forceinline__ bool gemm_has_work(const GemmOut& g, GemmRows m_tiles, int c) {
  if (g.all_work) return true;
  const long long U = (long long)(g.pair ? ((g.n_tiles + 1) >> 1) : g.n_tiles) * m_tiles.n * g.nkb, G = g.grid;
  return gemm_range_begin(c, U, G) < gemm_range_begin(c + 1, U, G);
}

constexpr int GEMM_FOLD_UNROLL = 8;  // slots loaded together (a tile rarely has more contributors)

// Two-phase read of a projection value: gemm_issue starts every load (output element and up to U
// partial slots) without consuming any of them, gemm_finish sums them in CTA order.  A kernel that
// needs several values issues all of them first, so the loads overlap instead of forming a chain
// of L2 round trips.  Tiles with more than U extra contributors take a (rare) loop in gemm_finish.
template <int U>
struct GemmPending {
  float raw;
  float q[U];
  GemmFold f;
};
template <int U>
struct GemmPending4 {
  float4 raw;
  float4 q[U];
  GemmFold f;
};

template <int U>
__device__ __forceinline__ GemmPending<U> gemm_issue(const GemmOut& g, GemmRows m_tiles, int m, int n) {
  GemmPending<U> p;
  p.raw = g.raw[(size_t)m * g.ld + n];
  p.f.c_next = 1; p.f.c_last = 0; p.f.off = 0;
  if (g.partial != nullptr) p.f = gemm_fold(g, m_tiles, m, n);
  const size_t slot = gemm_slot_stride(g);
#pragma unroll
  for (int j = 0; j < U; ++j) {
    const int c = p.f.c_next + j;
    p.q[j] = (c <= p.f.c_last && gemm_has_work(g, m_tiles, c)) ? __ldcg(g.partial + (size_t)c * slot + p.f.off) : 0.f;
  }
  return p;
}
template <int U>
__device__ __forceinline__ float gemm_finish(const GemmOut& g, GemmRows m_tiles, const GemmPending<U>& p) {
  float v = p.raw;
#pragma unroll
  for (int j = 0; j < U; ++j) v += p.q[j];
  const size_t slot = gemm_slot_stride(g);
  for (int c = p.f.c_next + U; c <= p.f.c_last; ++c)
    if (gemm_has_work(g, m_tiles, c)) v += __ldcg(g.partial + (size_t)c * slot + p.f.off);
  return v;
}
// Four consecutive columns n .. n+3 (n a multiple of 4: they share a tile and the slots' alignment).
template <int U>
__device__ __forceinline__ GemmPending4<U> gemm_issue4(const GemmOut& g, GemmRows m_tiles, int m, int n) {
  GemmPending4<U> p;
  p.raw = *reinterpret_cast<const float4*>(g.raw + (size_t)m * g.ld + n);
  p.f.c_next = 1; p.f.c_last = 0; p.f.off = 0;
  if (g.partial != nullptr) p.f = gemm_fold(g, m_tiles, m, n);
  const size_t slot = gemm_slot_stride(g);
#pragma unroll
  for (int j = 0; j < U; ++j) {
    const int c = p.f.c_next + j;
    p.q[j] = (c <= p.f.c_last && gemm_has_work(g, m_tiles, c))
                 ? __ldcg(reinterpret_cast<const float4*>(g.partial + (size_t)c * slot + p.f.off))
                 : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  return p;
}
template <int U>
__device__ __forceinline__ float4 gemm_finish4(const GemmOut& g, GemmRows m_tiles, const GemmPending4<U>& p) {
  float4 v = p.raw;
#pragma unroll
  for (int j = 0; j < U; ++j) { v.x += p.q[j].x; v.y += p.q[j].y; v.z += p.q[j].z; v.w += p.q[j].w; }
  const size_t slot = gemm_slot_stride(g);
  for (int c = p.f.c_next + U; c <= p.f.c_last; ++c) {
    if (!gemm_has_work(g, m_tiles, c)) continue;
    const float4 t = __ldcg(reinterpret_cast<const float4*>(g.partial + (size_t)c * slot + p.f.off));
    v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
  }
  return v;
}

// Two consecutive columns n, n+1 (n even) of row m, with the fold of a column of the same tile already
// computed: `doff` is n minus the column the fold was made for.  Lets a kernel that reads several column
// pairs of one tile (the two halves of a rotary pair) pay for the fold once.
__device__ __forceinline__ GemmFold gemm_fold_or_none(const GemmOut& g, GemmRows m_tiles, int m, int n) {
  GemmFold f;
  f.c_next = 1; f.c_last = 0; f.off = 0;
  if (g.partial != nullptr) f = gemm_fold(g, m_tiles, m, n);
  return f;
}
template <int U>
struct GemmPending2 {
  float2 raw;
  float2 q[U];
};
template <int U>
__device__ __forceinline__ GemmPending2<U> gemm_issue2(const GemmOut& g, GemmRows m_tiles, const GemmFold& f, int m, int n, int doff) {
  GemmPending2<U> p;
  p.raw = __ldcg(reinterpret_cast<const float2*>(g.raw + (size_t)m * g.ld + n));
  const size_t slot = gemm_slot_stride(g);
#pragma unroll
  for (int j = 0; j < U; ++j) {
    const int c = f.c_next + j;
    p.q[j] = (c <= f.c_last && gemm_has_work(g, m_tiles, c))
                 ? __ldcg(reinterpret_cast<const float2*>(g.partial + (size_t)c * slot + f.off + doff))
                 : make_float2(0.f, 0.f);
  }
  return p;
}
template <int U>
__device__ __forceinline__ float2 gemm_finish2(const GemmOut& g, GemmRows m_tiles, const GemmFold& f, int doff, const GemmPending2<U>& p) {
  float2 v = p.raw;
#pragma unroll
  for (int j = 0; j < U; ++j) { v.x += p.q[j].x; v.y += p.q[j].y; }
  const size_t slot = gemm_slot_stride(g);
  for (int c = f.c_next + U; c <= f.c_last; ++c) {
    if (!gemm_has_work(g, m_tiles, c)) continue;
    const float2 t = __ldcg(reinterpret_cast<const float2*>(g.partial + (size_t)c * slot + f.off + doff));
    v.x += t.x; v.y += t.y;
  }
  return v;
}

// ---- addresses first, data later ---------------------------------------------------------------
// The short kernels between two projections run once per layer with cold instruction caches, and what
// they execute AFTER their predecessor has finished is the step's critical path.  Where a value lives
// (output element, first partial slot, number of slots) depends only on launch constants, so a consumer
// works it out while it is still waiting; afterwards it only loads and adds.
struct GemmSrc {
  const float* raw;    // &raw[m][n]
  const float* part;   // the value's place in the first extra contributor's slot; slot j is at part + j * stride
  int n_extra;         // contributors other than the first (0 when the tile is not cut or on the CUDA-core path)
};
// Valid for launches where every CTA has work (all_work), which is every launch whose stream is at
// least as long as the grid; callers fall back to gemm_value* otherwise.
__device__ __forceinline__ GemmSrc gemm_src(const GemmOut& g, GemmRows m_tiles, int m, int n) {
  GemmSrc s;
  s.raw = g.raw + (size_t)m * g.ld + n;
  s.part = g.partial;
  s.n_extra = 0;
  if (g.partial != nullptr) {
    const GemmFold f = gemm_fold(g, m_tiles, m, n);
    s.part = g.partial + (size_t)f.c_next * gemm_slot_stride(g) + f.off;
    s.n_extra = f.c_last - f.c_next + 1;
  }
  return s;
}
// Keeps the compiler from sinking the address arithmetic below the wait.
__device__ __forceinline__ void gemm_src_pin(GemmSrc& s) {
  asm volatile("" : "+l"(s.raw), "+l"(s.part), "+r"(s.n_extra));
}
template <int U>
struct GemmData4 {
  float4 raw;
  float4 q[U];
};
template <int U>
struct GemmData2 {
  float2 raw;
  float2 q[U];
};
// `doff`: element offset from the column the source was made for (same tile, same row).
template <int U>
__device__ __forceinline__ GemmData4<U> gemm_load4(const GemmSrc& s, size_t stride, int doff = 0) {
  GemmData4<U> p;
  p.raw = __ldcg(reinterpret_cast<const float4*>(s.raw + doff));
#pragma unroll
  for (int j = 0; j < U; ++j)
    p.q[j] = j < s.n_extra ? __ldcg(reinterpret_cast<const float4*>(s.part + j * stride + doff)) : make_float4(0.f, 0.f, 0.f, 0.f);
  return p;
}
template <int U>
__device__ __forceinline__ float4 gemm_sum4(const GemmSrc& s, size_t stride, const GemmData4<U>& p, int doff = 0) {
  float4 v = p.raw;
#pragma unroll
  for (int j = 0; j < U; ++j) { v.x += p.q[j].x; v.y += p.q[j].y; v.z += p.q[j].z; v.w += p.q[j].w; }
  // more contributors than were loaded up front: the rest in batches of four loads (slot order is kept)
  for (int j = U; j < s.n_extra; j += 4) {
    float4 t[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      t[k] = j + k < s.n_extra ? __ldcg(reinterpret_cast<const float4*>(s.part + (j + k) * stride + doff)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int k = 0; k < 4; ++k) { v.x += t[k].x; v.y += t[k].y; v.z += t[k].z; v.w += t[k].w; }
  }
  return v;
}
template <int U>
__device__ __forceinline__ GemmData2<U> gemm_load2(const GemmSrc& s, size_t stride, int doff = 0) {
  GemmData2<U> p;
  p.raw = __ldcg(reinterpret_cast<const float2*>(s.raw + doff));
#pragma unroll
  for (int j = 0; j < U; ++j)
    p.q[j] = j < s.n_extra ? __ldcg(reinterpret_cast<const float2*>(s.part + j * stride + doff)) : make_float2(0.f, 0.f);
  return p;
}
template <int U>
__device__ __forceinline__ float2 gemm_sum2(const GemmSrc& s, size_t stride, const GemmData2<U>& p, int doff = 0) {
  float2 v = p.raw;
#pragma unroll
  for (int j = 0; j < U; ++j) { v.x += p.q[j].x; v.y += p.q[j].y; }
  for (int j = U; j < s.n_extra; ++j) {
    const float2 t = __ldcg(reinterpret_cast<const float2*>(s.part + j * stride + doff));
    v.x += t.x; v.y += t.y;
  }
  return v;
}

// One-shot forms.
__device__ __forceinline__ float gemm_value(const GemmOut& g, GemmRows m_tiles, int m, int n) {
  return gemm_finish(g, m_tiles, gemm_issue<GEMM_FOLD_UNROLL>(g, m_tiles, m, n));
}
template <int U = GEMM_FOLD_UNROLL>
__device__ __forceinline__ float4 gemm_value4(const GemmOut& g, GemmRows m_tiles, int m, int n) {
  return gemm_finish4(g, m_tiles, gemm_issue4<U>(g, m_tiles, m, n));
}

// Four consecutive columns with the fold worked out by the caller (a kernel that walks the rows of one row tile
// computes it once per tile: only the offset inside the slot, doff, changes from row to row).
template <int U>
struct GemmPending4f {
  float4 raw;
  float4 q[U];
};
template <int U>
__device__ __forceinline__ GemmPending4f<U> gemm_issue4f(const GemmOut& g, GemmRows m_tiles, const GemmFold& f, int m, int n, size_t doff) {
  GemmPending4f<U> p;
  p.raw = __ldcg(reinterpret_cast<const float4*>(g.raw + (size_t)m * g.ld + n));
  const size_t slot = gemm_slot_stride(g);
#pragma unroll
  for (int j = 0; j < U; ++j) {
    const int c = f.c_next + j;
    p.q[j] = (c <= f.c_last && gemm_has_work(g, m_tiles, c))
                 ? __ldcg(reinterpret_cast<const float4*>(g.partial + (size_t)c * slot + f.off + doff))
                 : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  return p;
}
template <int U>
__device__ __forceinline__ float4 gemm_finish4f(const GemmOut& g, GemmRows m_tiles, const GemmFold& f, size_t doff, const GemmPending4f<U>& p) {
  float4 v = p.raw;
#pragma unroll
  for (int j = 0; j < U; ++j) { v.x += p.q[j].x; v.y += p.q[j].y; v.z += p.q[j].z; v.w += p.q[j].w; }
  const size_t slot = gemm_slot_stride(g);
  for (int c = f.c_next + U; c <= f.c_last; ++c) {
    if (!gemm_has_work(g, m_tiles, c)) continue;
    const float4 t = __ldcg(reinterpret_cast<const float4*>(g.partial + (size_t)c * slot + f.off + doff));
    v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
  }
  return v;
}
// Rows [begin, end) of a kernel that splits M rows evenly over `parts` CTAs, part `i`.
__device__ __forceinline__ int gemm_rows_begin(int M, int parts, int i) { return (int)((long long)M * i / parts); }

}  // namespace rd

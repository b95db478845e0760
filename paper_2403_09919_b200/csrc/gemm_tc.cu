// Weight-streaming projection on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), bf16.
//
//   Y[m][n] = sum_k A[m][k] W[n][k]        A: [M][K] activations, W: [N][K] weights, both K-major
//
// At decode time M (packed tokens x batch) is small and the projection is bound by the weight
// stream, so the operands are swapped: the WEIGHT tile is the 128-row MMA "A" operand and the
// activations are the MMA "B" operand, N_mma = MT rows (a multiple of 16, at most 256).  The
// accumulator D[n][m] lives in TMEM: lane = weight row, column = activation row.
//
// Schedule: persistent, one CTA per SM, stream-K.  The work is the list of (row tile, weight tile,
// k-block) units, row tile slowest; tile = (128 weight rows) x (MT activation rows), k-block = 64
// columns; CTA c owns the contiguous unit range [c*U/G, (c+1)*U/G), so every SM streams the same
// number of weight bytes whatever the shape, and with several row tiles the CTAs of all row tiles
// walk the weight tiles abreast (a tile leaves device memory once).  With one row tile of at most
// 128 rows a unit is a PAIR of adjacent weight tiles sharing one activation box.  The rows of a
// launch are a device-side count: the box height, the MMA's N and the number of (equal) row tiles
// follow it (gemm_row_tiles).  No epilogue and no cross-CTA reduction happen here: the segment that
// holds a tile's first k-block stores its fp32 sums to the output, any other segment to the CTA's
// partial slot, and the consuming kernel folds them in CTA order (gemm_out.cuh).
//
// Roles: warp 0 = TMA producer (one or two 128x64 weight boxes and one activation box per stage),
// warp 1 = MMA issuer and TMEM owner, warps 2.. = epilogue (tcgen05.ld; one warp per TMEM lane quarter,
// or two that take every other group of 16 accumulator columns: see tc_threads).  Two TMEM accumulator buffers alternate so the epilogue of one segment overlaps the MMAs
// of the next; the smem ring (full/empty mbarriers) never drains between tiles.  The producer is a single
// thread, the MMA issuer a whole warp with one elected issuing lane: their loops carry their positions along and
// contain no division (a division by a run-time value per stage was what bounded the stream).
//
// Launches bounded by many rows run on CTA pairs instead (gemm_tc2_kernel below: tcgen05 cta_group::2, the
// two CTAs of a cluster share one activation box).
//
// Every mbarrier wait is bounded (one second); on expiry the CTA raises DEV_ERR_TIMEOUT in the
// status word, lets its copies land, frees its TMEM and exits; later launches see the flag and
// return at once.
#include <cuda.h>
#include <stdlib.h>

#include "gemm_out.cuh"
#include "pdl.cuh"
#include "rd_internal.cuh"

namespace rd {

namespace {

constexpr int TILE_N = 128;       // weight rows per tile (MMA M)
constexpr int TILE_K = 64;        // bf16 per k-block = one 128-byte swizzle row
constexpr int W_STAGE_BYTES = TILE_N * TILE_K * 2;
constexpr int MAX_STAGES = 16;    // ring slots the barrier block has room for
// Epilogue warps: one per tensor-memory lane quarter at decode size (fewer registers held beside the short kernels
// that share the SM), two per quarter -- each takes every other group of 16 accumulator columns -- where an
// accumulator buffer is wide: launches of more than 128 rows (up to 256 columns) and pair-mode launches of more than
// 64 rows (two tiles of up to 128 columns).  EW (4 or 8) is a template parameter.
__host__ __device__ constexpr int tc_threads(int ew) { return 64 + 32 * ew; }
constexpr unsigned long long WAIT_LIMIT_NS = 1000000000ull;

// Activation operand: one descriptor per box height, 16, 32, ..., 256 rows in m[0..15] (up to the launch's own
// height).  A launch that turns out to have a single row tile picks the smallest that holds the actual row count.
constexpr int ACT_MAPS = 16;
struct ActMaps {
  CUtensorMap m[ACT_MAPS];
};

struct TcParams {
  int N, K, nkb, n_tiles, mt, m_tiles_max, stages, tmem_cols;
  int ring_bytes;     // shared memory of the stage ring (at least stages full-height stages)
  const int32_t* m_total;
  float* raw;         // [M][ld_raw] fp32 output
  int ld_raw;
  float* partial;     // [gridDim.x][mt * 128]
  int32_t* status;
  unsigned long long* trace;  // 8 timestamps of this launch (see redrafter_trace_read) or nullptr
  ChainSync cs;       // counter hand-off with the launches before and after this one
  // 1: a unit is (pair of adjacent weight tiles, k-block): both tiles of a stage are multiplied by ONE activation
  // box, which halves what the activation operand costs an SM.  Single row tile only.
  int pair;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false when the CTA is aborting (this or another role gave up).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = globaltimer();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 255u) == 0u) {
      if (*abort_flag) return false;
      if (globaltimer() - t0 > WAIT_LIMIT_NS) {
        *abort_flag = 1;
        atomicOr(status, DEV_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

// Weight tiles are read once per step: they are marked evict-first so that the stream (hundreds of MB per
// layer) does not push the step's small working set -- residual stream, row tables, rotary table, norm gains'
// neighbours, partial sums -- out of the L2 between two uses.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y), "l"(pol)
      : "memory");
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, rows of 128 bytes, 8-row groups
// 1024 bytes apart (stride byte offset), descriptor version 1 (sm_100), leading offset unused (1).
__device__ __forceinline__ uint64_t umma_desc(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

template <int EW>
__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(32 * EW) : "memory"); }

// PAIR (one row tile of at most 128 rows): two adjacent weight tiles per stage share one activation box, and an
// accumulator buffer holds both tiles.  Measured and dropped: the same pairing at up to 256 rows and with several
// row tiles (a 256 x 256 output tile per unit).  Its two accumulators fill the tensor memory, so the epilogue no
// longer overlaps the next tile's MMAs, and that costs what the shared activation box saves.
template <bool PAIR, int EW>
__global__ void __launch_bounds__(tc_threads(EW), EW == 4 ? 4 : 2) gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w,
                                                                 const __grid_constant__ ActMaps maps_a,
                                                                 const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  pdl_launch_dependents();  // the next kernel may start its own prologue now
  if (p.trace && threadIdx.x == 0) { atomicMin(p.trace + 0, globaltimer()); }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // With a single row tile the work split does not depend on the row count, so the weight stream can
  // start before the preceding kernels have finished (they produce the activations and the row count).
  // Inside a chain the row count was written ahead of the chain's first launch and may be read at once,
  // so the same holds for any number of row tiles.
  const bool chained = p.cs.signal_ptr != nullptr;
  const bool early = (p.m_tiles_max == 1) || chained;
  if (!early) {
    if (threadIdx.x == 0) chain_wait_thread(p.cs);
    __syncthreads();
  }
  // Rows actually present: the activation box, the MMA's N and the epilogue shrink to the next multiple of 16.
  // Every byte of the activation operand is fetched once per weight tile, so at 48 rows it is more than a third
  // of what an SM has to pull in.  (A single row tile outside a chain keeps the full box: its row count is not
  // known yet.)
  GemmRows rows(1, p.mt);
  if (p.m_tiles_max > 1) rows = gemm_row_tiles(p.mt, p.m_tiles_max, *p.m_total);
  else if (chained) rows.rows = min(p.mt, max(16, (*p.m_total + 15) & ~15));
  const int m_tiles = rows.n;
  const long long G = gridDim.x;
  // unit = (row tile, weight tile or tile pair, k-block), row tile slowest: the CTAs of each row tile then walk the
  // weight tiles abreast of the other row tiles' CTAs, and a weight tile leaves device memory once for all of them
  const int n_wt = PAIR ? (p.n_tiles + 1) / 2 : p.n_tiles;
  const int n_groups = n_wt * m_tiles;
  const long long U = (long long)n_groups * p.nkb;
  const long long u0 = gemm_range_begin(blockIdx.x, U, G), u1 = gemm_range_begin(blockIdx.x + 1, U, G);
  const int mt_eff = rows.rows;   // several row tiles are equal: the fewest that hold the rows, each a multiple of 16 rows
  const CUtensorMap* map_a = &maps_a.m[(mt_eff >> 4) - 1];

  // ---- shared memory carve-up (stage buffers 1024-byte aligned for the 128-byte swizzle)
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t w_bytes = PAIR ? 2u * W_STAGE_BYTES : (uint32_t)W_STAGE_BYTES;
  const uint32_t ring_bytes = (uint32_t)p.ring_bytes;   // what the host reserved: p.stages stages of full height, or more
  // Outside the pair mode the ring is cut by the rows actually present: a launch laid out for 256-row tiles that
  // turns out to have 200 rows gets five stages instead of four, and the bytes in flight are what bounds the stream.
  const uint32_t stage_bytes = w_bytes + (uint32_t)(PAIR ? p.mt : mt_eff) * TILE_K * 2;
  const int n_stages = PAIR ? p.stages : min(MAX_STAGES, (int)(ring_bytes / stage_bytes));
  const uint32_t tx_bytes = w_bytes + (uint32_t)mt_eff * TILE_K * 2;   // arriving per stage
  const uint32_t bar_base = base + ring_bytes;  // 8-byte aligned
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (MAX_STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * MAX_STAGES + 2 + a); };
  uint8_t* misc = smem_raw + (bar_base - raw) + 8u * (2 * MAX_STAGES + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);
  volatile int* epi_ok = reinterpret_cast<volatile int*>(misc + 12);

  // iteration i of this CTA = unit u0 + i
  const uint32_t n_it = (uint32_t)(u1 - u0);
  const uint32_t pre = early ? min(n_it, (uint32_t)n_stages) : 0u;
  const uint64_t pol_w = l2_policy_evict_first();
  // Position of the producer in its unit range, advanced without divisions: the producer is a single thread, and
  // a division by a run-time value is a chain of a hundred dependent instructions -- several of them per stage
  // would bound the rate at which stages are issued.
  struct UnitPos {
    int g, m_tile, kb;     // weight tile (or tile pair), row tile, k-block
    uint32_t s, ph;        // ring slot and the parity of its current use
  };
  auto pos_at = [&](long long u) {
    UnitPos q;
    const int t = (int)(u / p.nkb);
    q.kb = (int)(u - (long long)t * p.nkb);
    q.m_tile = PAIR ? 0 : t / n_wt;
    q.g = t - q.m_tile * n_wt;
    q.s = 0; q.ph = 0;
    return q;
  };
  auto advance = [&](UnitPos& q) {
    if (++q.kb == p.nkb) {
      q.kb = 0;
      if (++q.g == n_wt) { q.g = 0; ++q.m_tile; }
    }
    if (++q.s == (uint32_t)n_stages) { q.s = 0; q.ph ^= 1u; }
  };
  auto issue_w = [&](const UnitPos& q) {
    const uint32_t dst = base + q.s * stage_bytes;
    mbar_expect_tx(full_bar(q.s), tx_bytes);
    if (PAIR) {
      // tiles 2g and 2g+1 (the second may lie past the matrix: the copy then delivers zeros)
      tma_load_2d_hint(dst, &map_w, full_bar(q.s), q.kb * TILE_K, (2 * q.g) * TILE_N, pol_w);
      tma_load_2d_hint(dst + W_STAGE_BYTES, &map_w, full_bar(q.s), q.kb * TILE_K, (2 * q.g + 1) * TILE_N, pol_w);
    } else {
      tma_load_2d_hint(dst, &map_w, full_bar(q.s), q.kb * TILE_K, q.g * TILE_N, pol_w);
    }
  };
  auto issue_a = [&](const UnitPos& q) {
    // one box of MT rows: the TMA unit's cost is per operation, not per byte, at these sizes
    tma_load_2d(base + q.s * stage_bytes + w_bytes, map_a, full_bar(q.s), q.kb * TILE_K, q.m_tile * mt_eff);
  };

  if (threadIdx.x == 0) {
    // The producer thread sets the barriers up and starts the weight stream at once: the weights of the
    // first ring-full of k-blocks depend on nothing in the step, and nothing of the CTA's remaining set-up
    // (tensor-memory allocation, the other roles' start) needs to come first.
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(map_a) : "memory");
    for (int s = 0; s < n_stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 32 * EW); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    UnitPos q = pos_at(u0);
    for (uint32_t i = 0; i < pre; ++i) { issue_w(q); advance(q); }
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"((uint32_t)p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0 && u0 < u1) {
      if (p.trace) atomicMax(p.trace + 7, globaltimer());   // last CTA ready to wait
      // An earlier launch of the step gave up on a wait: wind this one down through the roles' abort paths.  The
      // status word is requested BEFORE the wait (a load right after it would put an L2 round trip between the
      // dependency and the first activation copy); a time-out raised while this thread waits ends the wait itself.
      const int32_t status_before = *(volatile int32_t*)p.status;
      if (early) chain_wait_thread(p.cs);
      chain_fence_async_reads();  // the activations were written by ordinary stores of the preceding launch
      if (p.trace) { atomicMin(p.trace + 1, globaltimer()); atomicMax(p.trace + 2, globaltimer()); }   // dependency resolved
      if (status_before & DEV_ERR_TIMEOUT) *abort_flag = 1;
      UnitPos q = pos_at(u0);
      for (uint32_t i = 0; i < pre; ++i) { issue_a(q); advance(q); }
      bool ok = true;
      for (uint32_t i = pre; i < n_it; ++i) {
        if (!mbar_wait(empty_bar(q.s), q.ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
        issue_w(q);
        issue_a(q);
        advance(q);
      }
      if (!ok || *abort_flag) {  // give the copies already issued time to land before the CTA's shared memory is released
        const unsigned long long t0 = globaltimer();
        while (globaltimer() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    // The whole warp runs the loop (waits, descriptor arithmetic) and an elected lane issues: what is the same in
    // every lane stays in the uniform datapath, from which the MMA takes its descriptors; a lone active lane would
    // move each descriptor across per instruction (measured in the attention kernel: 80 against 39 ns per MMA issued).
    if (u0 < u1) {
      uint32_t leader;
      asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(leader));
      auto wait_warp = [&](uint32_t b, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag, p.status)) != 0;
      };
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(mt_eff >> 3) << 17) | ((uint32_t)(TILE_N >> 4) << 24);
      uint32_t seg = 0, s = 0, ph = 0;   // ring slot and parity, advanced without divisions
      bool ok = true;
      for (long long u = u0; u < u1 && ok; ++seg) {
        const int t = (int)(u / p.nkb), kb0 = (int)(u - (long long)t * p.nkb);
        const int kb1 = (int)min((long long)p.nkb, kb0 + (u1 - u));
        const uint32_t a = seg & 1u, aph = (seg >> 1) & 1u;
        if (!wait_warp(tempty_bar(a), aph ^ 1u)) { ok = false; break; }
        tc_fence_after();
        const uint32_t acc_cols = (uint32_t)p.mt * (PAIR ? 2u : 1u);   // columns of one accumulator buffer
        const uint32_t d_tmem = tmem_base + a * acc_cols;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!wait_warp(full_bar(s), ph)) { ok = false; break; }
          tc_fence_after();
          const uint64_t wdesc = umma_desc(base + s * stage_bytes);
          const uint64_t adesc = umma_desc(base + s * stage_bytes + w_bytes);
          if (leader) {
#pragma unroll
            for (int k = 0; k < TILE_K / 16; ++k)
              umma_bf16(d_tmem, wdesc + 2 * k, adesc + 2 * k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
            if (PAIR) {   // the stage's second weight tile against the same activation box
              const uint64_t wdesc2 = umma_desc(base + s * stage_bytes + W_STAGE_BYTES);
#pragma unroll
              for (int k = 0; k < TILE_K / 16; ++k)
                umma_bf16(d_tmem + (uint32_t)p.mt, wdesc2 + 2 * k, adesc + 2 * k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
            }
            umma_commit(empty_bar(s));  // the stage is free once these MMAs have read it
          }
          __syncwarp();
          if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1u; }
        }
        if (ok && leader) umma_commit(tfull_bar(a));
        __syncwarp();
        u += kb1 - kb0;
      }
      if (p.trace && leader) { atomicMin(p.trace + 3, globaltimer()); atomicMax(p.trace + 4, globaltimer()); }   // all MMAs issued
    }
  } else {
    // ===================== epilogue (warps 2..) =====================
    if (early) {                            // the row count comes from preceding kernels, and their readers of
      if (threadIdx.x == 64) chain_wait_thread(p.cs);   // this launch's output buffers must be done
      epi_bar_sync<EW>();
    }
    const int M = *p.m_total;
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int row = q * 32 + lane;          // weight row inside the tile
    const int et = threadIdx.x - 64;        // 0 .. (epilogue threads - 1)
    constexpr bool two_per_quarter = EW == 8;
    const int chunk_par = ((warp - 2) >> 2) & 1;   // which of the quarter's two warps: it takes every other 16 columns
    constexpr int chunk_step = two_per_quarter ? 32 : 16;
    uint32_t seg = 0;
    bool ok = true;
    for (long long u = u0; u < u1 && ok; ++seg) {
      const int t = (int)(u / p.nkb), kb0 = (int)(u - (long long)t * p.nkb);
      const int kb1 = (int)min((long long)p.nkb, kb0 + (u1 - u));
      const int m_tile = PAIR ? 0 : t / n_wt, grp = t - m_tile * n_wt;
      const int n_tile0 = PAIR ? 2 * grp : grp;
      const int m_base = m_tile * mt_eff;
      const int c_end = min(mt_eff, ((M - m_base) + 15) & ~15);   // accumulator columns that hold rows of the launch
      const uint32_t a = seg & 1u, aph = (seg >> 1) & 1u;
      // one thread does the bounded wait and tells the others, so that all 128 take the same branch
      if (et == 0) *epi_ok = mbar_wait(tfull_bar(a), aph, abort_flag, p.status) ? 1 : 0;
      epi_bar_sync<EW>();
      if (!*epi_ok) { ok = false; break; }
      tc_fence_after();
      const uint32_t acc_cols = (uint32_t)p.mt * (PAIR ? 2u : 1u);
      const size_t slot_floats = (size_t)acc_cols * TILE_N;
      for (int sub = 0; sub < (PAIR ? 2 : 1); ++sub) {
        const int n = (n_tile0 + sub) * TILE_N + row;
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * acc_cols + (uint32_t)sub * (uint32_t)p.mt;
        float* my_partial = p.partial + (size_t)blockIdx.x * slot_floats + (size_t)sub * p.mt * TILE_N;
        for (int c0 = two_per_quarter ? 16 * (chunk_par ^ (sub & 1)) : 0; c0 < c_end; c0 += chunk_step) {
          uint32_t r[16];
          tmem_ld16(taddr + c0, r);
          if (kb0 == 0) {
            // this segment holds the tile's first k-block: its sums go to the output
            if (n < p.N) {
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const int m = m_base + c0 + j;
                if (m < M) p.raw[(size_t)m * p.ld_raw + n] = __uint_as_float(r[j]);
              }
            }
          } else {
            // the range starts inside this tile: at most one such segment per CTA
#pragma unroll
            for (int j = 0; j < 16; ++j) my_partial[(size_t)(c0 + j) * TILE_N + row] = __uint_as_float(r[j]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(tempty_bar(a));  // the accumulator may be overwritten
      u += kb1 - kb0;
    }
  }

  // ---- teardown: everyone meets, then the allocating warp frees the TMEM columns
  tc_fence_before();
  __syncthreads();
  if (p.trace && threadIdx.x == 0) { atomicMin(p.trace + 5, globaltimer()); atomicMax(p.trace + 6, globaltimer()); }   // CTA done
  chain_exit(p.cs);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
  }
}


// ---------------------------------------------------------------------------------------------
// CTA pairs (tcgen05 cta_group::2) for launches of more than 128 rows
// ---------------------------------------------------------------------------------------------
// Beyond 128 rows a stage holds one weight tile (16 KB) and an activation box of up to 256 rows (32 KB): an SM
// pulls in two to three times as many activation bytes (from L2) as weight bytes, and that intake, not the
// weight stream or the tensor pipe, bounds the projection.  Here the two CTAs of a cluster work as one: each loads
// ITS weight tile of a pair of adjacent tiles and HALF of the activation box, and one MMA of shape 256 x N x 16
// issued by the leader multiplies both weight tiles by the whole box (the hardware reads each half from the CTA
// that holds it).  Each CTA's tensor memory receives the accumulator of its own weight tile, so the epilogue and
// the output layout are those of the pair mode above with "CTA" read as "cluster": units run over (row tile,
// pair of weight tiles, k-block), cluster c owns [c*U/C, (c+1)*U/C), a partial slot holds the two tiles of a pair.
//
// Barriers.  full[s]: in the leader, completed by the bytes of both CTAs' copies (the peer's copies name the
// leader's barrier).  empty[s] and tfull[a]: one in each CTA, the leader's MMA thread commits to both.
// tempty[a]: in the leader, one arrival per epilogue warp of either CTA.  Before a CTA leaves, its producer waits
// until the commits to its own empty barriers have landed and the cluster meets once more, so that no signal is
// sent to shared memory that has been given back.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Copy into this CTA's shared memory; the bytes are counted on `bar`, which may lie in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
// Arrives on one barrier (an address of the cluster's shared-memory window) once the MMAs issued so far are done.
__device__ __forceinline__ void umma_commit_pair(uint32_t cluster_bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_bar) : "memory");
}

template <int EW>
__global__ void __launch_bounds__(tc_threads(EW), EW == 4 ? 4 : 2) gemm_tc2_kernel(const __grid_constant__ CUtensorMap map_w,
                                                                  const __grid_constant__ ActMaps maps_a,   // box heights 8, 16, ..., 128
                                                                  const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  pdl_launch_dependents();
  if (p.trace && threadIdx.x == 0) { atomicMin(p.trace + 0, globaltimer()); }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();        // 0: leader (issues the MMAs), 1: peer
  const uint32_t cluster = cluster_id_x();
  const bool chained = p.cs.signal_ptr != nullptr;
  const bool early = (p.m_tiles_max == 1) || chained;
  if (!early) {
    if (threadIdx.x == 0) chain_wait_thread(p.cs);
    __syncthreads();
  }
  GemmRows rows(1, p.mt);
  if (p.m_tiles_max > 1) rows = gemm_row_tiles(p.mt, p.m_tiles_max, *p.m_total);
  else if (chained) rows.rows = min(p.mt, max(16, (*p.m_total + 15) & ~15));
  const int m_tiles = rows.n;
  const long long C = gridDim.x >> 1;             // clusters
  const int n_wt = (p.n_tiles + 1) / 2;           // pairs of weight tiles
  const int n_groups = n_wt * m_tiles;
  const long long U = (long long)n_groups * p.nkb;
  const long long u0 = gemm_range_begin(cluster, U, C), u1 = gemm_range_begin(cluster + 1, U, C);
  const int mt_eff = rows.rows, half = mt_eff >> 1;   // rows of a row tile; rows of it this CTA loads
  const CUtensorMap* map_a = &maps_a.m[(half >> 3) - 1];

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t a_stage_bytes = (uint32_t)(p.mt >> 1) * TILE_K * 2;   // reserved
  const uint32_t stage_bytes = (uint32_t)W_STAGE_BYTES + a_stage_bytes;
  const uint32_t tx_bytes = 2u * ((uint32_t)W_STAGE_BYTES + (uint32_t)half * TILE_K * 2);   // both CTAs' copies of a stage
  const uint32_t bar_base = base + p.stages * stage_bytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (p.stages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * p.stages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * p.stages + 2 + a); };
  uint8_t* misc = smem_raw + (bar_base - raw) + 8u * (2 * p.stages + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);
  volatile int* epi_ok = reinterpret_cast<volatile int*>(misc + 12);

  const uint32_t n_it = (uint32_t)(u1 - u0);
  const uint32_t pre = early ? min(n_it, (uint32_t)p.stages) : 0u;
  const uint64_t pol_w = l2_policy_evict_first();
  struct UnitPos {
    int g, m_tile, kb;
    uint32_t s, ph;
  };
  auto pos_at = [&](long long u) {
    UnitPos q;
    const int t = (int)(u / p.nkb);
    q.kb = (int)(u - (long long)t * p.nkb);
    q.m_tile = t / n_wt;
    q.g = t - q.m_tile * n_wt;
    q.s = 0; q.ph = 0;
    return q;
  };
  auto advance = [&](UnitPos& q) {
    if (++q.kb == p.nkb) {
      q.kb = 0;
      if (++q.g == n_wt) { q.g = 0; ++q.m_tile; }
    }
    if (++q.s == (uint32_t)p.stages) { q.s = 0; q.ph ^= 1u; }
  };
  // the bytes of both CTAs are counted on the leader's barrier; the leader announces them
  auto issue_w = [&](const UnitPos& q) {
    if (rank == 0) mbar_expect_tx(full_bar(q.s), tx_bytes);
    // tile 2g + rank (the odd one may lie past the matrix: the copy then delivers zeros)
    tma_load_2d_pair_hint(base + q.s * stage_bytes, &map_w, map_to_cta(full_bar(q.s), 0), q.kb * TILE_K,
                          (2 * q.g + (int)rank) * TILE_N, pol_w);
  };
  auto issue_a = [&](const UnitPos& q) {
    tma_load_2d_pair(base + q.s * stage_bytes + W_STAGE_BYTES, map_a, map_to_cta(full_bar(q.s), 0), q.kb * TILE_K,
                     q.m_tile * mt_eff + (int)rank * half);
  };

  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(map_a) : "memory");
    for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * EW); }   // one arrival per epilogue warp of either CTA
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"((uint32_t)p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  // both CTAs' barriers exist before either sends a signal to the other
  tc_fence_before();
  __syncwarp();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ===================== TMA producer (one per CTA) =====================
    if (lane == 0 && u0 < u1) {
      UnitPos q = pos_at(u0);
      for (uint32_t i = 0; i < pre; ++i) { issue_w(q); advance(q); }
      if (p.trace) atomicMax(p.trace + 7, globaltimer());
      const int32_t status_before = *(volatile int32_t*)p.status;
      if (early) chain_wait_thread(p.cs);
      chain_fence_async_reads();
      if (p.trace) { atomicMin(p.trace + 1, globaltimer()); atomicMax(p.trace + 2, globaltimer()); }
      if (status_before & DEV_ERR_TIMEOUT) *abort_flag = 1;
      q = pos_at(u0);
      for (uint32_t i = 0; i < pre; ++i) { issue_a(q); advance(q); }
      bool ok = true;
      for (uint32_t i = pre; i < n_it; ++i) {
        if (!mbar_wait(empty_bar(q.s), q.ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
        issue_w(q);
        issue_a(q);
        advance(q);
      }
      // the leader's commits to this CTA's empty barriers must have landed before its shared memory is given back
      if (ok) {
        if (n_it < (uint32_t)p.stages) {
          for (uint32_t s = 0; s < n_it && ok; ++s) ok = mbar_wait(empty_bar(s), 0u, abort_flag, p.status);
        } else {
          for (int j = 0; j < p.stages && ok; ++j) {
            ok = mbar_wait(empty_bar(q.s), q.ph ^ 1u, abort_flag, p.status);
            if (++q.s == (uint32_t)p.stages) { q.s = 0; q.ph ^= 1u; }
          }
        }
      }
      if (!ok || *abort_flag) {
        const unsigned long long t0 = globaltimer();
        while (globaltimer() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer (leader CTA only) =====================
    // (whole warp, elected lane: see gemm_tc_kernel)
    if (u0 < u1 && rank == 0) {
      uint32_t leader;
      asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(leader));
      auto wait_warp = [&](uint32_t b, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag, p.status)) != 0;
      };
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(mt_eff >> 3) << 17) | ((uint32_t)((2 * TILE_N) >> 4) << 24);
      uint32_t seg = 0, s = 0, ph = 0;
      bool ok = true;
      for (long long u = u0; u < u1 && ok; ++seg) {
        const int t = (int)(u / p.nkb), kb0 = (int)(u - (long long)t * p.nkb);
        const int kb1 = (int)min((long long)p.nkb, kb0 + (u1 - u));
        const uint32_t a = seg & 1u, aph = (seg >> 1) & 1u;
        if (!wait_warp(tempty_bar(a), aph ^ 1u)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * (uint32_t)p.mt;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!wait_warp(full_bar(s), ph)) { ok = false; break; }
          tc_fence_after();
          const uint64_t wdesc = umma_desc(base + s * stage_bytes);
          const uint64_t adesc = umma_desc(base + s * stage_bytes + W_STAGE_BYTES);
          if (leader) {
#pragma unroll
            for (int k = 0; k < TILE_K / 16; ++k)
              umma_bf16_pair(d_tmem, wdesc + 2 * k, adesc + 2 * k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
            umma_commit_pair(empty_bar(s));                  // this CTA's stage
            umma_commit_pair(map_to_cta(empty_bar(s), 1));   // and the peer's
          }
          __syncwarp();
          if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; }
        }
        if (ok && leader) {
          umma_commit_pair(tfull_bar(a));
          umma_commit_pair(map_to_cta(tfull_bar(a), 1));
        }
        __syncwarp();
        u += kb1 - kb0;
      }
      if (p.trace && leader) { atomicMin(p.trace + 3, globaltimer()); atomicMax(p.trace + 4, globaltimer()); }
      // the epilogue warps' arrivals for the last accumulators (the peer's come over the cluster) land before the end
      for (uint32_t k = 0; k < 2u && k < seg && ok; ++k) {
        const uint32_t sg = seg - 1 - k;
        ok = wait_warp(tempty_bar(sg & 1u), (sg >> 1) & 1u);
      }
    }
  } else {
    // ===================== epilogue (warps 2.. of both CTAs) =====================
    if (early) {
      if (threadIdx.x == 64) chain_wait_thread(p.cs);
      epi_bar_sync<EW>();
    }
    const int M = *p.m_total;
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const int et = threadIdx.x - 64;
    constexpr bool two_per_quarter = EW == 8;
    const int chunk_par = ((warp - 2) >> 2) & 1;
    constexpr int chunk_step = two_per_quarter ? 32 : 16;
    const uint32_t tempty_leader0 = map_to_cta(tempty_bar(0), 0), tempty_leader1 = map_to_cta(tempty_bar(1), 0);
    uint32_t seg = 0;
    bool ok = true;
    for (long long u = u0; u < u1 && ok; ++seg) {
      const int t = (int)(u / p.nkb), kb0 = (int)(u - (long long)t * p.nkb);
      const int kb1 = (int)min((long long)p.nkb, kb0 + (u1 - u));
      const int m_tile = t / n_wt, grp = t - m_tile * n_wt;
      const int m_base = m_tile * mt_eff;
      const int c_end = min(mt_eff, ((M - m_base) + 15) & ~15);
      const uint32_t a = seg & 1u, aph = (seg >> 1) & 1u;
      if (et == 0) *epi_ok = mbar_wait(tfull_bar(a), aph, abort_flag, p.status) ? 1 : 0;
      epi_bar_sync<EW>();
      if (!*epi_ok) { ok = false; break; }
      tc_fence_after();
      const int n = (2 * grp + (int)rank) * TILE_N + row;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * (uint32_t)p.mt;
      // slot of the cluster: [tile 2g | tile 2g + 1], each [mt][128]
      float* my_partial = p.partial + ((size_t)cluster * 2 + rank) * (size_t)p.mt * TILE_N;
      for (int c0 = two_per_quarter ? 16 * chunk_par : 0; c0 < c_end; c0 += chunk_step) {
        uint32_t r[16];
        tmem_ld16(taddr + c0, r);
        if (kb0 == 0) {
          if (n < p.N) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int m = m_base + c0 + j;
              if (m < M) p.raw[(size_t)m * p.ld_raw + n] = __uint_as_float(r[j]);
            }
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) my_partial[(size_t)(c0 + j) * TILE_N + row] = __uint_as_float(r[j]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(a ? tempty_leader1 : tempty_leader0);
      u += kb1 - kb0;
    }
  }

  // ---- teardown: the pair meets (no signal is under way to either CTA's shared memory), then the tensor memory goes back
  tc_fence_before();
  __syncthreads();
  if (p.trace && threadIdx.x == 0) { atomicMin(p.trace + 5, globaltimer()); atomicMax(p.trace + 6, globaltimer()); }
  chain_exit(p.cs);
  __syncwarp();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
  }
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// Tensor map of a row-major bf16 matrix [rows][cols] with a (box_rows x 64) box and 128-byte swizzle.
int tc_make_map(void* out_map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return -1;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {TILE_K, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn((CUtensorMap*)out_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return (int)r;
}

int tc_weight_box_rows() { return TILE_N; }

// Weight bytes the CTAs of the most recent launch (of this host thread) request BEFORE their dependency wait: the
// first ring-full of stages.  Measurement aid: an in-place rate must not count them against the time after the wait.
static thread_local double g_last_prefetch_bytes = 0.0;
double tc_last_prefetch_bytes() { return g_last_prefetch_bytes; }

// Activation rows per tile for a launch whose row count is at most m_max.
int tc_pick_mt(int m_max) {
  // One row tile up to 256 rows.  Beyond that the tiles are 256 rows: the bound is a host-side one (batch x rows per
  // sequence) and the actual count is often below 256, in which case the kernel runs a single tile after all.
  if (m_max > 256) return 256;
  const int mt = (m_max + 15) / 16 * 16;
  return mt < 16 ? 16 : mt;
}

size_t tc_partial_floats(int grid, int mt) { return (size_t)grid * mt * TILE_N * 2; }   // room for pair mode

// Launch helpers for the CTA-pair kernel: clusters of two CTAs along x.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pairs(bool ordered, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  prefer_max_shared(reinterpret_cast<const void*>(kernel));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = ordered ? 1 : 2;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(std::forward<Args>(args))...);
}

// smem_limit_out: dynamic shared memory a projection CTA may ask for.  pairs_out: CTA pairs (clusters of two) of
// the pair kernel that can be resident at once with that much shared memory, 0 when it cannot be used.
cudaError_t tc_prepare(int* smem_limit_out, int* pairs_out) {
  int dev = 0, lim = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&lim, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  cudaFuncAttributes fa;
  e = cudaFuncGetAttributes(&fa, gemm_tc_kernel<false, 4>);
  if (e != cudaSuccess) return e;
  lim -= (int)fa.sharedSizeBytes;  // the opt-in limit covers static + dynamic shared memory
  e = cudaFuncSetAttribute(gemm_tc_kernel<false, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<false, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<true, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<true, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc2_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
  if (smem_limit_out) *smem_limit_out = lim;
  if (pairs_out) {
    *pairs_out = 0;
    if (e == cudaSuccess) {
      int sms = 0;
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)(sms & ~1));
      cfg.blockDim = dim3(tc_threads(8));
      cfg.dynamicSmemBytes = (size_t)lim;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      int n = 0;
      const cudaError_t oe = cudaOccupancyMaxActiveClusters(&n, gemm_tc2_kernel<8>, &cfg);
      if (oe == cudaSuccess) *pairs_out = n;
      else cudaGetLastError();
    }
  }
  return e;
}

// Whether a launch bounded by m_max rows runs on CTA pairs (gemm_tc2_kernel): a bound of at least min_rows (the
// caller's threshold), at least one pair of weight tiles, and pairs for (nearly) every SM resident at once.  The
// activation descriptors of such a launch have box heights 8, 16, ..., mt / 2.
bool tc_use_pairs(int m_max, int N, int grid, int pairs, int min_rows) {
  return m_max >= min_rows && m_max > 16 && N > TILE_N && pairs > 0 && 2 * pairs >= grid - 4;
}

// The CTA-pair kernel: `pairs` clusters of two CTAs.  map_a: box heights 8, 16, ..., mt / 2.
static cudaError_t launch_gemm_tc2(const void* map_w, const void* const map_a[16], int N, int K, const int32_t* m_total, int m_max,
                                   float* raw, int ld_raw, float* partial, int32_t* status, int pairs, int smem_limit,
                                   unsigned long long* trace, GemmOut* out_desc, Chain* chain, cudaStream_t st) {
  TcParams p;
  p.N = N; p.K = K; p.nkb = (K + TILE_K - 1) / TILE_K; p.n_tiles = (N + TILE_N - 1) / TILE_N;
  p.mt = tc_pick_mt(m_max);
  p.m_tiles_max = (m_max + p.mt - 1) / p.mt;
  p.pair = 1;
  const long long n_units = (long long)((p.n_tiles + 1) / 2) * p.nkb;
  if (out_desc) {
    // for the consumers a cluster is what a CTA is in pair mode: units over pairs of tiles, a slot holds both tiles
    out_desc->raw = raw; out_desc->partial = partial; out_desc->ld = ld_raw; out_desc->nkb = p.nkb;
    out_desc->n_tiles = p.n_tiles; out_desc->mt = p.mt; out_desc->grid = pairs; out_desc->m_tiles_max = p.m_tiles_max;
    out_desc->all_work = (n_units >= pairs) ? 1 : 0;
    out_desc->pair = 1;
    out_desc->small32 = ((n_units * p.m_tiles_max + 1) * pairs < (1ll << 31)) ? 1 : 0;
  }
  const int stage_bytes = W_STAGE_BYTES + (p.mt / 2) * TILE_K * 2;
  const int overhead = 1024 + 8 * (2 * 16 + 4) + 64;
  int stages = (smem_limit - overhead) / stage_bytes;
  if (stages > 16) stages = 16;
  if (stages < 2) return cudaErrorInvalidConfiguration;
  p.stages = stages;
  int cols = 32;
  while (cols < 2 * p.mt) cols <<= 1;
  p.tmem_cols = cols;
  p.m_total = m_total; p.raw = raw; p.ld_raw = ld_raw; p.partial = partial; p.status = status; p.trace = trace;
  const bool first = chain && chain->enabled && chain->prev_ptr == nullptr;
  p.cs = chain ? chain->link((unsigned)(2 * pairs)) : ChainSync{nullptr, 0u, nullptr, status, nullptr};
  const size_t smem = (size_t)stages * stage_bytes + overhead;
  {
    const long long per_cta = (n_units * p.m_tiles_max) / pairs;   // units of a cluster (each CTA loads one weight tile per unit)
    g_last_prefetch_bytes = (p.m_tiles_max == 1 || chain) ? 2.0 * pairs * (double)(per_cta < stages ? per_cta : stages) * W_STAGE_BYTES : 0.0;
  }
  ActMaps am;
  for (int i = 0; i < ACT_MAPS; ++i) am.m[i] = *(const CUtensorMap*)(map_a[i] ? map_a[i] : map_a[0]);
  launch_pairs(first, gemm_tc2_kernel<8>, 2 * pairs, tc_threads(8), smem, st, *(const CUtensorMap*)map_w, am, p);
  return cudaGetLastError();
}

cudaError_t launch_gemm_tc(const void* map_w, const void* const map_a[16], int N, int K, const int32_t* m_total, int m_max,
                           float* raw, int ld_raw, float* partial, int32_t* status, int grid, int pairs, int smem_limit,
                           unsigned long long* trace, GemmOut* out_desc, Chain* chain, int pair, cudaStream_t st) {
  if (tc_use_pairs(m_max, N, grid, pairs, 0))   // the caller passes pairs = 0 below its row threshold
    return launch_gemm_tc2(map_w, map_a, N, K, m_total, m_max, raw, ld_raw, partial, status, pairs < grid / 2 ? pairs : grid / 2,
                           smem_limit, trace, out_desc, chain, st);
  TcParams p;
  p.N = N; p.K = K; p.nkb = (K + TILE_K - 1) / TILE_K; p.n_tiles = (N + TILE_N - 1) / TILE_N;
  p.mt = tc_pick_mt(m_max > 0 ? m_max : 1);
  p.m_tiles_max = m_max > 0 ? (m_max + p.mt - 1) / p.mt : 1;
  static const int pair_ok = getenv("RD_TC_PAIR") ? atoi(getenv("RD_TC_PAIR")) : 1;   // tuning toggle
  p.pair = (pair && pair_ok && p.m_tiles_max == 1 && p.mt <= 128 && p.n_tiles >= 2) ? 1 : 0;
  const long long n_units = (long long)(p.pair ? (p.n_tiles + 1) / 2 : p.n_tiles) * p.nkb;
  if (out_desc) {
    out_desc->raw = raw; out_desc->partial = partial; out_desc->ld = ld_raw; out_desc->nkb = p.nkb;
    out_desc->n_tiles = p.n_tiles; out_desc->mt = p.mt; out_desc->grid = grid; out_desc->m_tiles_max = p.m_tiles_max;
    out_desc->all_work = (n_units >= grid) ? 1 : 0;
    out_desc->pair = p.pair ? 1 : 0;
    out_desc->small32 = ((n_units * p.m_tiles_max + 1) * grid < (1ll << 31)) ? 1 : 0;
  }
  if (m_max <= 0) return cudaSuccess;
  const int stage_bytes = W_STAGE_BYTES * (p.pair ? 2 : 1) + p.mt * TILE_K * 2;
  const int overhead = 1024 + 8 * (2 * 16 + 4) + 64;
  // Skinny launches (the decode step) take 168 KB at most -- four stages of a pair of weight tiles plus the
  // activation box -- and leave the rest of the SM's shared memory to the small kernels that run between
  // projections, so that this kernel can become resident, and start its weight stream, while they are still
  // running.  (Measured: a fifth stage does not pay.)
  static const int cap_kb = getenv("RD_TC_SMEM_KB") ? atoi(getenv("RD_TC_SMEM_KB")) : 168;   // tuning toggles
  const int budget = p.mt <= 64 ? (smem_limit < cap_kb * 1024 ? smem_limit : cap_kb * 1024) : smem_limit;
  int stages = (budget - overhead) / stage_bytes;
  if (stages > 16) stages = 16;
  if (stages < 2) return cudaErrorInvalidConfiguration;
  p.stages = stages;
  // outside the pair mode the kernel cuts the ring itself, by the rows present: it gets everything the budget allows
  p.ring_bytes = p.pair ? stages * stage_bytes : ((budget - overhead) & ~1023);
  int cols = 32;
  while (cols < 2 * p.mt * (p.pair ? 2 : 1)) cols <<= 1;
  p.tmem_cols = cols;
  p.m_total = m_total; p.raw = raw; p.ld_raw = ld_raw; p.partial = partial; p.status = status; p.trace = trace;
  // the first launch of a chain starts after everything before it has completed (see launch_ordered)
  const bool first = chain && chain->enabled && chain->prev_ptr == nullptr;
  p.cs = chain ? chain->link((unsigned)grid) : ChainSync{nullptr, 0u, nullptr, status, nullptr};
  const size_t smem = (size_t)p.ring_bytes + overhead;
  {
    // (outside the pair mode the kernel may fit more stages than `stages` when few rows are present: a lower bound)
    const long long per_cta = (n_units * p.m_tiles_max) / grid;
    g_last_prefetch_bytes = (p.m_tiles_max == 1 || chain) ? (double)grid * (double)(per_cta < stages ? per_cta : stages) *
                                                            W_STAGE_BYTES * (p.pair ? 2 : 1) : 0.0;
  }
  ActMaps am;
  for (int i = 0; i < ACT_MAPS; ++i) am.m[i] = *(const CUtensorMap*)(map_a[i] ? map_a[i] : map_a[0]);
  if (p.pair) {
    if (p.mt > 64) {   // two tiles of up to 128 columns per accumulator buffer: the epilogue on eight warps
      if (first) launch_ordered(gemm_tc_kernel<true, 8>, grid, tc_threads(8), smem, st, *(const CUtensorMap*)map_w, am, p);
      else launch_pdl(gemm_tc_kernel<true, 8>, grid, tc_threads(8), smem, st, *(const CUtensorMap*)map_w, am, p);
    } else {
      if (first) launch_ordered(gemm_tc_kernel<true, 4>, grid, tc_threads(4), smem, st, *(const CUtensorMap*)map_w, am, p);
      else launch_pdl(gemm_tc_kernel<true, 4>, grid, tc_threads(4), smem, st, *(const CUtensorMap*)map_w, am, p);
    }
  } else {
    if (p.mt > 128) {
      if (first) launch_ordered(gemm_tc_kernel<false, 8>, grid, tc_threads(8), smem, st, *(const CUtensorMap*)map_w, am, p);
      else launch_pdl(gemm_tc_kernel<false, 8>, grid, tc_threads(8), smem, st, *(const CUtensorMap*)map_w, am, p);
    } else {
      if (first) launch_ordered(gemm_tc_kernel<false, 4>, grid, tc_threads(4), smem, st, *(const CUtensorMap*)map_w, am, p);
      else launch_pdl(gemm_tc_kernel<false, 4>, grid, tc_threads(4), smem, st, *(const CUtensorMap*)map_w, am, p);
    }
  }
  return cudaGetLastError();
}

}  // namespace rd

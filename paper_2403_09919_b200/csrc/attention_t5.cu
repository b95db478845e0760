// Tree-masked / causal attention on the 5th-generation tensor cores for launches with many rows per sequence
// (Sections 3.3, 3.4): head dimension 128, bf16 operands, fp32 accumulation in tensor memory.
//
// One CTA = (head, sequence, tile of 128 of its rows).  Keys come in chunks of 128:
//   S = Q K^T   tcgen05.mma, A = Q tile (128 rows x 128 dims, K-major in shared memory, converted once from the fp32
//               rows the rotary kernel wrote), B = K chunk (128 keys x 128 dims, K-major, straight from the cache by
//               TMA), D = S in tensor memory (two buffers, so the next chunk's scores are computed during this
//               chunk's softmax);
//   softmax     four threads per query row (= TMEM lane), a quarter of the chunk's keys each: scale, mask, running
//               maximum and sum in registers (base 2), P written back to tensor memory as packed bf16 (two buffers, so
//               a chunk's probabilities are formed while the previous chunk's P V runs);
//   correction  two more threads per query row scale O in tensor memory when the row's maximum moved, between the previous
//               chunk's P V and this one's -- off the softmax threads' path, which publish the factor before they
//               exponentiate (measured: with the rescale inside the softmax loop a chunk took 1.7 us, 0.5 us of it
//               waiting for the previous P V);
//   O += P V    tcgen05.mma with A = P read from tensor memory (8 packed columns per 16 keys), B = V chunk as it lies
//               in the cache ([key][dim], i.e. MN-major for this product: leading byte offset = one 64-dim box of the
//               chunk, stride byte offset = 8 keys, 2048 bytes per 16 keys).
// Tensor memory: columns 0..255 the two score buffers, 256..383 O, 384..511 the two P buffers.
// Roles: warp 0 lane 0 = TMA producer (K and V rings of two chunks), warp 1 lane 0 = MMA issuer (warp 1 owns the tensor
// memory; the whole warp runs the issue loop and an elected lane issues, see there),
// warps 2..17 = softmax and output, warps 18..25 = correction.  Every wait is bounded (one second): on expiry the CTA raises
// DEV_ERR_TIMEOUT, lets its copies land, frees its tensor memory and leaves.
//
// The chunk's keys past a row's extent are masked by selection, never by arithmetic, and their V rows are multiplied by
// exact zeros: the cache must hold finite values everywhere (it is cleared once when the handle is created).
#include <cuda.h>
#include <stdio.h>

#include "pdl.cuh"
#include "rd_internal.cuh"

namespace rd {

namespace {

constexpr int T5_ROWS = 128;      // query rows per CTA (one TMEM lane each)
constexpr int T5_KEYS = 128;      // keys per chunk
constexpr int T5_HD = 128;
constexpr int T5_STAGES = 2;      // K and V chunks in flight
constexpr int T5_PARTS = 4;        // softmax threads per query row (each a part of the chunk's keys and of the head dimensions)
constexpr int T5_SOFT = 128 * T5_PARTS;
constexpr int T5_CORR_PARTS = 2;  // correction threads per query row (each half of the head dimensions)
constexpr int T5_CORR = 128 * T5_CORR_PARTS;
constexpr int T5_THREADS = 64 + T5_SOFT + T5_CORR;
constexpr uint32_t T5_BLOCK = 128 * 128;            // bytes of one 64-column block of 128 rows (128 B per row)
constexpr uint32_t T5_TILE = 2 * T5_BLOCK;          // Q tile, K chunk, V chunk, P tile: 32 KB each
constexpr unsigned long long T5_WAIT_NS = 1000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long now_ns() {
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
  const unsigned long long t0 = now_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 255u) == 0u) {
      if (*abort_flag) return false;
      if (now_ns() - t0 > T5_WAIT_NS) {
        *abort_flag = 1;
        atomicOr(status, DEV_ERR_TIMEOUT);
        return false;
      }
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
// K-major operand, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// MN-major operand, 128-byte swizzle: 64 MN-elements (128 bytes) per row of a block, 8 K-rows 1024 bytes apart, the next
// 64 MN-elements one block (T5_BLOCK bytes) further.
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(T5_BLOCK >> 4) << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
// A operand read from tensor memory (lane = row, packed bf16 pairs along the columns).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 32 consecutive columns of this thread's lane; the caller waits once after issuing all its loads (a load followed
// at once by its wait costs a few hundred nanoseconds each time).
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, float* r) {
  uint32_t u[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, "
      "%20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]), "=r"(u[9]),
        "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]), "=r"(u[17]), "=r"(u[18]),
        "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]),
        "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr));
#pragma unroll
  for (int j = 0; j < 32; ++j) r[j] = __uint_as_float(u[j]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, "
      "%19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(__float_as_uint(r[0])), "r"(__float_as_uint(r[1])), "r"(__float_as_uint(r[2])), "r"(__float_as_uint(r[3])),
      "r"(__float_as_uint(r[4])), "r"(__float_as_uint(r[5])), "r"(__float_as_uint(r[6])), "r"(__float_as_uint(r[7])),
      "r"(__float_as_uint(r[8])), "r"(__float_as_uint(r[9])), "r"(__float_as_uint(r[10])), "r"(__float_as_uint(r[11])),
      "r"(__float_as_uint(r[12])), "r"(__float_as_uint(r[13])), "r"(__float_as_uint(r[14])), "r"(__float_as_uint(r[15])),
      "r"(__float_as_uint(r[16])), "r"(__float_as_uint(r[17])), "r"(__float_as_uint(r[18])), "r"(__float_as_uint(r[19])),
      "r"(__float_as_uint(r[20])), "r"(__float_as_uint(r[21])), "r"(__float_as_uint(r[22])), "r"(__float_as_uint(r[23])),
      "r"(__float_as_uint(r[24])), "r"(__float_as_uint(r[25])), "r"(__float_as_uint(r[26])), "r"(__float_as_uint(r[27])),
      "r"(__float_as_uint(r[28])), "r"(__float_as_uint(r[29])), "r"(__float_as_uint(r[30])), "r"(__float_as_uint(r[31]))
      : "memory");
}
__device__ __forceinline__ void tmem_st16_u32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void soft_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(T5_SOFT) : "memory"); }
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Measurement build (-DRD_T5_STAMPS, never the shipped library): the CTA of head 0 / sequence 0 / first row tile of the
// 41st launch records %globaltimer at the steps of chunks 2..9 in one softmax thread, the MMA warp and one correction
// thread, and prints the timeline when it is done.
#ifdef RD_T5_STAMPS
__device__ unsigned long long g_t5_st[3][8][8];
__device__ int g_t5_launch = 0;
#define T5_STAMP(on, role, c, i) do { if ((on) && (c) >= 2 && (c) < 10) g_t5_st[role][(c) - 2][i] = now_ns(); } while (0)
#else
#define T5_STAMP(on, role, c, i) do { } while (0)
#endif

struct T5Params {
  const float* qkv;            // [M][3d] fp32, Q rotated in place by the rotary kernel
  __nv_bfloat16* out;          // [M][d]
  RowTables rt;
  const int32_t* seq_off;
  const int32_t* seq_order;    // the launch's sequences, longest key extent first, or nullptr (index order)
  Dims dm;
  int row_tiles;               // 128-row tiles per sequence (bound)
  int32_t* status;
  ChainSync cs;
};

__global__ void __launch_bounds__(T5_THREADS, 1)
    attention_t5_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const T5Params p) {
  extern __shared__ uint8_t smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // ---- shared memory carve-up (operand tiles 1024-byte aligned for the 128-byte swizzle)
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);                 // generic pointer to the same place
  const uint32_t sQ = base, sK = sQ + T5_TILE, sV = sK + T5_STAGES * T5_TILE;
  const uint32_t bar0 = sV + T5_STAGES * T5_TILE;
  enum { Q_FULL = 0, K_FULL = 1, V_FULL = 3, K_EMPTY = 5, V_EMPTY = 7, S_FULL = 9, S_EMPTY = 11, P_FULL = 13, P_EMPTY = 15, X_FULL = 17, C_FULL = 18, O_READY = 20, N_BARS = 22 };
  auto bar = [&](int i) { return bar0 + 8u * i; };
  uint8_t* misc = gen + (bar0 - base) + 8u * 32;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);
  int32_t* s_ncache = reinterpret_cast<int32_t*>(misc + 16);              // [T5_ROWS]
  float* s_red = reinterpret_cast<float*>(misc + 16 + T5_ROWS * 4);       // [2][PARTS][T5_ROWS] row maxima of the parts, [PARTS][T5_ROWS] their sums
  float* s_corr = s_red + 3 * T5_PARTS * T5_ROWS;                         // [2][T5_ROWS] factor by which chunk c scales the row's running output
  uint32_t* s_mask = reinterpret_cast<uint32_t*>(s_corr + 2 * T5_ROWS);   // [T5_ROWS][MW]

  // Tensor memory first (512 columns: two score buffers and the output), before the dependents may start.
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  chain_begin(p.cs);
  // Launched inside a chain, the kernel may read before its wait whatever the launches ahead of the chain wrote: the
  // row tables and the tree mask.  Q and this pass's K/V come from the kernel right before it.
  const bool early = p.cs.signal_ptr != nullptr;
  if (!early) chain_wait_cta(p.cs);
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    mbar_init(bar(Q_FULL), T5_SOFT / 32);   // one arrival per softmax warp (256 arrivals on one barrier would serialise)
    for (int s = 0; s < T5_STAGES; ++s) {
      mbar_init(bar(K_FULL + s), 1); mbar_init(bar(V_FULL + s), 1);
      mbar_init(bar(K_EMPTY + s), 1); mbar_init(bar(V_EMPTY + s), 1);
      mbar_init(bar(S_FULL + s), 1); mbar_init(bar(S_EMPTY + s), T5_SOFT / 32);
    }
    for (int s = 0; s < 2; ++s) { mbar_init(bar(P_FULL + s), T5_SOFT / 32); mbar_init(bar(P_EMPTY + s), 1); }
    mbar_init(bar(X_FULL), T5_SOFT / 32);
    // (two of each, by chunk parity: the softmax and correction warps can be a chunk ahead of the warp that waits --
    // a single barrier could then complete two phases between two looks of its waiter, which reads as "not yet")
    for (int s = 0; s < 2; ++s) { mbar_init(bar(C_FULL + s), 4); mbar_init(bar(O_READY + s), T5_CORR / 32); }   // C_FULL: the four warps that hold part 0 of their rows
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  const Dims& dm = p.dm;
  const int h = blockIdx.x;
  // the tiles of a sequence are handed out last first: without a tree mask a later tile has more keys to walk, and
  // the longest CTAs should not be the last to start
  // ... and the sequences longest first (the row tables' order, when the launch has one)
  const int bi = blockIdx.y / p.row_tiles, rb = p.row_tiles - 1 - (blockIdx.y - bi * p.row_tiles);
  const int b = p.seq_order ? p.seq_order[bi] : bi;
  const int seq_row0 = p.seq_off[b], seq_rows = p.seq_off[b + 1] - seq_row0;
  const int row0 = seq_row0 + rb * T5_ROWS;
  const int nrows = min(T5_ROWS, seq_rows - rb * T5_ROWS);   // <= 0: nothing to do for this tile (same for all roles)
  const bool tree = p.rt.mask != nullptr;
  const int MW = dm.MW;
  int kext = 0, nc_min = 0, tree_base = 0;
  if (nrows > 0) {
    const int nc_first = p.rt.n_cache[row0], nc_last = p.rt.n_cache[row0 + nrows - 1];
    tree_base = nc_first;
    kext = min(tree ? tree_base + seq_rows : nc_last, dm.max_ctx);
    nc_min = tree ? tree_base : nc_first;   // every valid row attends at least the keys below this
  }
  const int n_chunks = (kext + T5_KEYS - 1) / T5_KEYS;
#ifdef RD_T5_STAMPS
  if (threadIdx.x == 0)
    *reinterpret_cast<volatile int*>(misc + 8) = (blockIdx.x == 0 && blockIdx.y == (unsigned)(p.row_tiles - 1)) ? atomicAdd(&g_t5_launch, 1) : -1;
#endif
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
#ifdef RD_T5_STAMPS
  const bool dbg_on = *reinterpret_cast<volatile int*>(misc + 8) == 40 && n_chunks >= 10;
#endif
  const uint32_t tmem = *tmem_slot;   // columns [0,128) and [128,256): scores, [256,384): output

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0 && n_chunks > 0) {
      const int key_row0 = (b * dm.H + h) * dm.max_ctx;   // first row of this (sequence, head) in the cache plane
      bool ok = true;
      auto load_k = [&](int c) {
        const int s = c & 1;
        mbar_expect_tx(bar(K_FULL + s), T5_TILE);
        tma_load_2d(sK + s * T5_TILE, &map_k, bar(K_FULL + s), 0, key_row0 + c * T5_KEYS);
        tma_load_2d(sK + s * T5_TILE + T5_BLOCK, &map_k, bar(K_FULL + s), 64, key_row0 + c * T5_KEYS);
      };
      auto load_v = [&](int c) {
        const int s = c & 1;
        mbar_expect_tx(bar(V_FULL + s), T5_TILE);
        tma_load_2d(sV + s * T5_TILE, &map_v, bar(V_FULL + s), 0, key_row0 + c * T5_KEYS);
        tma_load_2d(sV + s * T5_TILE + T5_BLOCK, &map_v, bar(V_FULL + s), 64, key_row0 + c * T5_KEYS);
      };
      // Chunks that hold only keys of earlier passes (tree: the context; causal: everything before the slot of the
      // sequence's first row of this pass) do not depend on the launch before this one: requested before the wait.
      int pre_k = 0, pre_v = 0;
      if (early) {
        const int const_keys = tree ? tree_base : p.rt.n_cache[seq_row0] - 1;
        while (pre_k < 2 && pre_k < n_chunks && (pre_k + 1) * T5_KEYS <= const_keys) load_k(pre_k++);
        if (pre_k > 0) { load_v(0); pre_v = 1; }
        chain_wait_thread(p.cs);
      }
      chain_fence_async_reads();   // this pass's keys and values were written with ordinary stores by the rotary kernel
      // K runs two chunks ahead (its slot is free once the scores of the chunk before last exist), V one (its slot is
      // free once the chunk before last has been added to the output, which is later): the order of the requests follows
      // the order in which the slots come free, so that no request waits behind one whose slot is still in use.
      for (int c = pre_k; c < 2 && c < n_chunks; ++c) load_k(c);
      for (int c = 0; c < n_chunks && ok; ++c) {
        const int s = c & 1;
        const uint32_t ph = (c >> 1) & 1;
        if (c >= pre_v) {
          if (c >= T5_STAGES) {
            if (!mbar_wait(bar(V_EMPTY + s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
          }
          load_v(c);
        }
        if (c + 2 < n_chunks) {
          if (!mbar_wait(bar(K_EMPTY + s), ph, abort_flag, p.status)) { ok = false; break; }   // Q K^T of chunk c is done
          load_k(c + 2);
        }
      }
      if (!ok || *abort_flag) {  // give the copies already issued time to land before the CTA's shared memory is released
        const unsigned long long t0 = now_ns();
        while (now_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    // The WHOLE warp runs this loop (waits, descriptor arithmetic), and one elected lane issues: values that are the
    // same in every lane stay in the uniform datapath, from which the MMA instruction takes its descriptors.  With a
    // single active lane the compiler cannot know that and moves every descriptor across per MMA -- a dozen extra
    // instructions in a warp that gets only every seventh issue slot beside the softmax warps (measured: 80 ns per
    // MMA issued against 39 ns this way; the MMA itself takes 35 ns).
    if (n_chunks > 0) {
      uint32_t leader;
      asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(leader));
      const uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(T5_KEYS >> 3) << 17) | ((uint32_t)(T5_ROWS >> 4) << 24);
      const uint32_t idesc_pv = idesc_qk | (1u << 16);   // second operand MN-major; N = 128 head dimensions
      auto wait_warp = [&](uint32_t b, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag, p.status)) != 0;
      };
      bool ok = wait_warp(bar(Q_FULL), 0);
      // descriptors once; a k-step adds a constant to the start-address field (16-byte units)
      const uint64_t q_desc = desc_kmajor(sQ);
      auto issue_qk = [&](int c) {
        const int s = c & 1;
        const uint32_t ph = (c >> 1) & 1;
        if (!wait_warp(bar(K_FULL + s), ph)) return false;
        T5_STAMP(dbg_on && leader, 1, c - 1, 0);
        if (!wait_warp(bar(S_EMPTY + s), ph ^ 1u)) return false;
        T5_STAMP(dbg_on && leader, 1, c - 1, 1);
        tc_fence_after();
        const uint64_t kd = desc_kmajor(sK + (uint32_t)s * T5_TILE);
        const uint32_t d = tmem + (uint32_t)s * T5_KEYS;
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < T5_HD / 16; ++kk) {
            const uint64_t off = (uint64_t)(((uint32_t)(kk >> 2) * T5_BLOCK + (uint32_t)(kk & 3) * 32u) >> 4);
            umma_bf16(d, q_desc + off, kd + off, idesc_qk, kk > 0 ? 1u : 0u);
          }
          umma_commit(bar(S_FULL + s));
          umma_commit(bar(K_EMPTY + s));
        }
        __syncwarp();
        return true;
      };
      if (ok) ok = issue_qk(0);
      for (int c = 0; c < n_chunks && ok; ++c) {
        const int s = c & 1;
        const uint32_t ph = (c >> 1) & 1;
        if (c + 1 < n_chunks) {
          if (!issue_qk(c + 1)) { ok = false; break; }
        }
        T5_STAMP(dbg_on && leader, 1, c, 2);
        // (the probabilities come last of the three: the other two waits are out of the way when they arrive)
        if (!wait_warp(bar(V_FULL + s), ph)) { ok = false; break; }
        T5_STAMP(dbg_on && leader, 1, c, 3);
        // the running output has been scaled to this chunk's reference maximum (correction warps)
        if (!wait_warp(bar(O_READY + (c & 1)), ph)) { ok = false; break; }
        T5_STAMP(dbg_on && leader, 1, c, 4);
        if (!wait_warp(bar(P_FULL + (c & 1)), ph)) { ok = false; break; }
        T5_STAMP(dbg_on && leader, 1, c, 5);
        tc_fence_after();
        const uint64_t vd = desc_mnmajor(sV + (uint32_t)s * T5_TILE);
        const uint32_t pa = tmem + 3u * T5_KEYS + (uint32_t)(c & 1) * (T5_KEYS / 2);
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < T5_KEYS / 16; ++kk) {
            // P from tensor memory: buffer c & 1, 16 keys = 8 packed columns further per step; V: 16 keys = 2048 bytes further
            umma_bf16_ts(tmem + 2u * T5_KEYS, pa + (uint32_t)kk * 8u, vd + (uint64_t)(kk * 128), idesc_pv, (c > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(bar(V_EMPTY + s));
          umma_commit(bar(P_EMPTY + (c & 1)));   // this P buffer may be overwritten and O is up to date through chunk c
        }
        __syncwarp();
        T5_STAMP(dbg_on && leader, 1, c, 6);
      }
    }
  } else if (warp < 2 + T5_SOFT / 32) {
    // ===================== softmax and output (warps 2..17) =====================
    // Four threads per query row (= TMEM lane): a warp may only touch the lane quarter (warp id mod 4), so warps w,
    // w + 4, w + 8 and w + 12 share a quarter; each takes a quarter of a chunk's keys and of the output dimensions.
    const int q4 = warp & 3;                      // TMEM lane quarter this warp may access
    const int hf = (warp - 2) >> 2;               // which part of the chunk's keys / of the head dimensions
    const int t = q4 * 32 + lane;                 // row inside the tile
    const int st = threadIdx.x - 64;              // 0..255 (for cooperative loads)
    const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
    const bool valid = t < nrows;
    if (n_chunks > 0) {
      // row tables and mask do not depend on the preceding kernel
      if (st < T5_ROWS) s_ncache[st] = st < nrows ? p.rt.n_cache[row0 + st] : 0;
      if (tree)
        for (int idx = st; idx < T5_ROWS * MW; idx += T5_SOFT) {
          const int r = idx / MW, wd = idx - r * MW;
          s_mask[idx] = r < nrows ? p.rt.mask[((size_t)b * dm.NMAX + rb * T5_ROWS + r) * MW + wd] : 0u;
        }
      if (st == 0 && early) chain_wait_thread(p.cs);
      soft_bar_sync();
      // Q tile -> bf16, K-major swizzled (16-byte chunk c of row r lands at chunk c ^ (r & 7) of its 128-byte line).
      // A warp converts two rows per pass: lane l takes the eight dimensions of chunk l & 15 of row 2i + (l >> 4), so a
      // pass reads two contiguous 512-byte rows.
      {
        const int cq = lane & 15;
        constexpr int WROWS = T5_ROWS / (T5_SOFT / 32);   // rows per warp
        const int wrow0 = (warp - 2) * WROWS;
#pragma unroll 4
        for (int i = 0; i < WROWS / 2; ++i) {
          const int r = wrow0 + 2 * i + (lane >> 4);
          uint4 v = make_uint4(0u, 0u, 0u, 0u);
          if (r < nrows) {
            const float* q = p.qkv + (size_t)(row0 + r) * 3 * dm.d + h * T5_HD + cq * 8;
            const float4 a = __ldcg(reinterpret_cast<const float4*>(q)), bq = __ldcg(reinterpret_cast<const float4*>(q + 4));
            v = make_uint4(pack_bf16(a.x, a.y), pack_bf16(a.z, a.w), pack_bf16(bq.x, bq.y), pack_bf16(bq.z, bq.w));
          }
          *reinterpret_cast<uint4*>(gen + (size_t)(cq >> 3) * T5_BLOCK + r * 128 + (((cq & 7) ^ (r & 7)) << 4)) = v;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(Q_FULL));
      }
      const int nc_row = s_ncache[t];
      const float scale2 = rsqrtf((float)T5_HD) * 1.4426950408889634f;   // 1/sqrt(hd) * log2(e)
      float m_run = -INFINITY, l_run = 0.f;       // l_run: this thread's half of the row's sum
      bool ok = true;
      // Every thread waits on the barrier itself (bounded) and the warp takes one decision, so that the warp-wide
      // tensor-memory instructions stay converged.  A warp that gives up stops arriving on the barriers the others wait
      // for; they give up in turn (the abort flag is checked in every bounded wait).
      auto wait_all = [&](uint32_t b, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag, p.status)) != 0;
      };
      // exchange between the two threads of a row: every warp arrives once it has written, then waits for all eight
      uint32_t x_phase = 0;
      auto exchange = [&]() {
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(X_FULL));
        const bool r = wait_all(bar(X_FULL), x_phase);
        x_phase ^= 1u;
        return r;
      };
      // Which of this thread's 32 keys [k0, k0 + 32) may row t attend?  One bit per key, formed from whole words: the
      // keys below the row's extent, with the bits of the tree part (keys tree_base .. tree_base + seq_rows) replaced
      // by the row's mask bits.  (Evaluated per key, with a shared-memory load each, the two masked chunks of a tile
      // took 2.3 us apiece.)  Masking is by selection, never arithmetic: masked scores may be anything.
      auto visible_word = [&](int k0) {
        const int n = nc_row - k0;
        uint32_t w = n >= 32 ? 0xffffffffu : (n <= 0 ? 0u : ((1u << n) - 1u));
        if (tree) {
          const int tb0 = k0 - tree_base;   // mask bit of key k0; negative when the chunk starts inside the context
          if (tb0 > -32 && tb0 < seq_rows) {
            const int j_lo = max(0, -tb0), j_hi = min(32, seq_rows - tb0);   // bit positions that lie in the tree part
            const uint32_t range = (j_hi >= 32 ? 0xffffffffu : ((1u << j_hi) - 1u)) & ~((1u << j_lo) - 1u);
            uint32_t bits;
            if (tb0 >= 0) {
              const int wd = tb0 >> 5;
              const uint32_t lo = s_mask[t * MW + wd], hi = (wd + 1 < MW) ? s_mask[t * MW + wd + 1] : 0u;
              bits = __funnelshift_r(lo, hi, (uint32_t)(tb0 & 31));
            } else {
              bits = s_mask[t * MW] << (-tb0);
            }
            w = (w & ~range) | (bits & range);
          }
        }
        return w;
      };
      constexpr int HALF = T5_KEYS / T5_PARTS;   // keys (and output dimensions) of this thread
      static_assert(HALF == 32, "visible_word forms one 32-bit word per thread and chunk");
      for (int c = 0; c < n_chunks; ++c) {
        const int s = c & 1;
        const uint32_t ph = (c >> 1) & 1;
        const int k0 = c * T5_KEYS + hf * HALF;   // first key of this thread's half
#ifdef RD_T5_STAMPS
        const bool dbg_me = dbg_on && threadIdx.x == 64;
#endif
        T5_STAMP(dbg_me, 0, c, 0);
        ok = wait_all(bar(S_FULL + s), ph);
        if (!ok) break;
        T5_STAMP(dbg_me, 0, c, 1);
        tc_fence_after();
        const uint32_t s_addr = tmem + lane_addr + (uint32_t)s * T5_KEYS + (uint32_t)hf * HALF;
        const bool all_visible = c * T5_KEYS + T5_KEYS <= nc_min;
        // ---- this thread's 64 scores into registers (one wait for both loads); the score buffer is then free for the
        // chunk after next
        float sc[HALF];
#pragma unroll
        for (int g = 0; g < HALF / 32; ++g) tmem_ld32_nowait(s_addr + g * 32, sc + g * 32);
        tmem_ld_wait();
        T5_STAMP(dbg_me, 0, c, 2);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(S_EMPTY + s));
        // ---- maximum of the visible ones (masked scores become -inf by selection)
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (all_visible) {
#pragma unroll
          for (int j = 0; j < HALF; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], sc[j]);
        } else {
          const uint32_t vw = visible_word(k0);
#pragma unroll
          for (int j = 0; j < HALF; ++j) {
            sc[j] = ((vw >> j) & 1u) ? sc[j] : -INFINITY;
            mx4[j & 3] = fmaxf(mx4[j & 3], sc[j]);
          }
        }
        // the softmax runs in base 2: 1/sqrt(hd) * log2(e) is folded into one multiply-add per score
        float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale2;   // scale2 > 0
        // the row's maximum over all parts
        s_red[((c & 1) * T5_PARTS + hf) * T5_ROWS + t] = mx;
        T5_STAMP(dbg_me, 0, c, 3);
        ok = exchange();
        if (!ok) break;
        T5_STAMP(dbg_me, 0, c, 4);
        // this chunk's P buffer is free once the P V of the chunk before last has read it
        if (c >= 2) {
          ok = wait_all(bar(P_EMPTY + (c & 1)), ph ^ 1u);
          if (!ok) break;
          tc_fence_after();
        }
#pragma unroll
        for (int q = 0; q < T5_PARTS; ++q) mx = fmaxf(mx, s_red[((c & 1) * T5_PARTS + q) * T5_ROWS + t]);
        T5_STAMP(dbg_me, 0, c, 5);
        const float m_new = fmaxf(m_run, mx);
        const float corr = (m_new == -INFINITY) ? 1.f : fast_exp2(m_run - m_new);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        // the factor for the running output goes to the correction warps at once: they scale O (once the previous
        // chunk's P V has completed) while this thread forms the probabilities.  All parts of a row compute the same
        // factor; part 0 publishes it.
        if (hf == 0) {
          s_corr[(c & 1) * T5_ROWS + t] = corr;
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(C_FULL + (c & 1)));
        }
        // ---- probabilities -> tensor memory (packed bf16: key pair (2j, 2j + 1) of this thread's keys in column j of its
        // part of buffer c & 1), row sum
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < HALF; ++j) { sc[j] = fast_exp2(fmaf(sc[j], scale2, -m_use)); sum4[j & 3] += sc[j]; }   // 2^(-inf) = 0
        {
          uint32_t pk[HALF / 2];
#pragma unroll
          for (int j = 0; j < HALF / 2; ++j) pk[j] = pack_bf16(sc[2 * j], sc[2 * j + 1]);
          tmem_st16_u32(tmem + lane_addr + 3u * T5_KEYS + (uint32_t)(c & 1) * (T5_KEYS / 2) + (uint32_t)hf * (HALF / 2), pk);
        }
        l_run = l_run * corr + ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
        m_run = m_new;
        T5_STAMP(dbg_me, 0, c, 6);
        tmem_st_wait();   // P is in tensor memory
        T5_STAMP(dbg_me, 0, c, 7);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(P_FULL + (c & 1)));
      }
      // ---- output: O / l, each thread its 64 dimensions
      if (ok) {
        s_red[(2 * T5_PARTS + hf) * T5_ROWS + t] = l_run;
        ok = exchange();
      }
      if (ok) ok = wait_all(bar(P_EMPTY + ((n_chunks - 1) & 1)), (uint32_t)(((n_chunks - 1) >> 1) & 1));
      if (ok) {
        tc_fence_after();
        float l_row = 0.f;
#pragma unroll
        for (int q = 0; q < T5_PARTS; ++q) l_row += s_red[(2 * T5_PARTS + q) * T5_ROWS + t];
        const float inv = l_row > 0.f ? 1.f / l_row : 0.f;
        const uint32_t o_addr = tmem + lane_addr + 2u * T5_KEYS + (uint32_t)hf * (T5_HD / T5_PARTS);
        __nv_bfloat16* o = p.out + (size_t)(row0 + (valid ? t : 0)) * dm.d + h * T5_HD + hf * (T5_HD / T5_PARTS);
#pragma unroll 1
        for (int g = 0; g < T5_HD / T5_PARTS / 32; ++g) {
          float ov[32];
          tmem_ld32_nowait(o_addr + g * 32, ov);
          tmem_ld_wait();
          if (valid) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
              *reinterpret_cast<uint4*>(o + g * 32 + q * 8) =
                  make_uint4(pack_bf16(ov[q * 8] * inv, ov[q * 8 + 1] * inv), pack_bf16(ov[q * 8 + 2] * inv, ov[q * 8 + 3] * inv),
                             pack_bf16(ov[q * 8 + 4] * inv, ov[q * 8 + 5] * inv), pack_bf16(ov[q * 8 + 6] * inv, ov[q * 8 + 7] * inv));
          }
        }
      }
    }
  } else {
    // ===================== correction (warps 18..25) =====================
    // Two threads per query row, half of the head dimensions each: O *= 2^(m_old - m_new) in tensor memory whenever a
    // row's reference maximum moved, between the previous chunk's P V and this one's.  Off the softmax threads' path:
    // they publish the factor before they exponentiate, and the MMA issuer waits for O_READY before the chunk's P V.
    const int q4 = warp & 3;
    const int hf = (warp - 2 - T5_SOFT / 32) >> 2;
    const int t = q4 * 32 + lane;
    const uint32_t o_addr = tmem + ((uint32_t)(q4 * 32) << 16) + 2u * T5_KEYS + (uint32_t)hf * (T5_HD / T5_CORR_PARTS);
    auto wait_all = [&](uint32_t b, uint32_t parity) {
      return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag, p.status)) != 0;
    };
    for (int c = 0; c < n_chunks; ++c) {
      if (!wait_all(bar(C_FULL + (c & 1)), (uint32_t)((c >> 1) & 1))) break;
#ifdef RD_T5_STAMPS
      const bool dbg_c = dbg_on && warp == 2 + T5_SOFT / 32 && lane == 0;
#endif
      T5_STAMP(dbg_c, 2, c, 0);
      const float corr = s_corr[(c & 1) * T5_ROWS + t];
      if (c > 0 && __any_sync(0xffffffffu, corr != 1.f)) {
        // O has to be complete through the previous chunk first
        if (!wait_all(bar(P_EMPTY + ((c - 1) & 1)), (uint32_t)(((c - 1) >> 1) & 1))) break;
        T5_STAMP(dbg_c, 2, c, 1);
        tc_fence_after();
        float ov[T5_HD / T5_CORR_PARTS];
#pragma unroll
        for (int g = 0; g < T5_HD / T5_CORR_PARTS / 32; ++g) tmem_ld32_nowait(o_addr + g * 32, ov + g * 32);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < T5_HD / T5_CORR_PARTS; ++j) ov[j] *= corr;
#pragma unroll
        for (int g = 0; g < T5_HD / T5_CORR_PARTS / 32; ++g) tmem_st32(o_addr + g * 32, ov + g * 32);
        tmem_st_wait();
        tc_fence_before();
      }
      T5_STAMP(dbg_c, 2, c, 2);
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(O_READY + (c & 1)));
    }
  }

  // a tile without rows still waits for its predecessor before it reports completion (the hand-off's ordering is
  // transitive only through CTAs that have seen the launch before them complete)
  if (n_chunks == 0 && threadIdx.x == 0) chain_wait_thread(p.cs);
  // ---- teardown: everyone meets, then the allocating warp frees the tensor memory
  tc_fence_before();
  __syncthreads();
  chain_exit(p.cs);
#ifdef RD_T5_STAMPS
  if (dbg_on && threadIdx.x == 0) {
    const unsigned long long t0 = g_t5_st[0][0][0];
    auto rel = [&](int role, int c, int i) { return (long long)(g_t5_st[role][c][i] - t0); };
    printf("t5 stamps (ns from the softmax thread's start of chunk 2), %d chunks, %d rows\n", n_chunks, nrows);
    for (int c = 0; c < 8; ++c)
      printf("c%d soft: start %lld Sfull %lld ld %lld max %lld xchg %lld Pempty %lld exp %lld st %lld | mma: Kfull(c+1) %lld Sempty %lld "
             "qk_issued %lld Vfull %lld Oready %lld Pfull %lld pv_issued %lld | corr: Cfull %lld PVdone %lld done %lld\n",
             c + 2, rel(0, c, 0), rel(0, c, 1), rel(0, c, 2), rel(0, c, 3), rel(0, c, 4), rel(0, c, 5), rel(0, c, 6), rel(0, c, 7),
             rel(1, c, 0), rel(1, c, 1), rel(1, c, 2), rel(1, c, 3), rel(1, c, 4), rel(1, c, 5), rel(1, c, 6), rel(2, c, 0),
             rel(2, c, 1), rel(2, c, 2));
  }
#endif
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

size_t t5_smem_bytes(int MW) {
  return 1024 + (size_t)(1 + 2 * T5_STAGES) * T5_TILE + 8 * 32 + 16 + T5_ROWS * 4 + 3 * T5_PARTS * T5_ROWS * 4 + 2 * T5_ROWS * 4 + (size_t)T5_ROWS * MW * 4 + 64;
}

}  // namespace

int attn_t5_rows_per_block() { return T5_ROWS; }
bool attn_t5_supported(int hd) { return hd == T5_HD; }

cudaError_t attn_t5_prepare(int hd, int MW) {
  if (hd != T5_HD) return cudaSuccess;
  return cudaFuncSetAttribute(attention_t5_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t5_smem_bytes(MW));
}

// map_k / map_v: tensor maps of the layer's K and V planes ([sequences * heads * max_ctx rows][128 dims], box 64 x 128).
// grid (H, sequences * row_tiles): row_tiles tiles of 128 rows cover the longest sequence of the launch.
cudaError_t launch_attention_t5(const void* map_k, const void* map_v, const float* qkv, void* out, const RowTables& rt,
                                const int32_t* seq_off, const int32_t* seq_order, const Dims& dm, int n_seq, int row_tiles,
                                int32_t* status, Chain* chain,
                                cudaStream_t st) {
  if (dm.hd != T5_HD) return cudaErrorInvalidValue;
  dim3 grid(dm.H, n_seq * row_tiles);
  T5Params p;
  p.qkv = qkv; p.out = (__nv_bfloat16*)out; p.rt = rt; p.seq_off = seq_off; p.seq_order = seq_order; p.dm = dm; p.row_tiles = row_tiles; p.status = status;
  p.cs = chain ? chain->link(grid.x * grid.y) : ChainSync{nullptr, 0u, nullptr, status, nullptr};
  launch_pdl(attention_t5_kernel, grid, T5_THREADS, t5_smem_bytes(dm.MW), st, *(const CUtensorMap*)map_k, *(const CUtensorMap*)map_v, p);
  return cudaGetLastError();
}

}  // namespace rd

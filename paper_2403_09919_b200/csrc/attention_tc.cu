// Tree-masked attention for the bf16 path (Sections 3.3, 3.4): KV tiles staged through shared
// memory with 128-bit asynchronous copies (double buffered), scores and P*V on the tensor cores
// (mma.sync m16n8k16: the work per tile is far too small for tcgen05), online softmax in fp32.
//
// One CTA = (head, sequence, tile of 16 of its rows, key split).  The four warps share the 16 rows
// and split every 64-key chunk four ways (16 keys each), each with its own running softmax; they
// are combined through shared memory at the end, so a decode step with a few dozen rows per
// sequence needs no cross-CTA merge at all and still spreads over heads x row tiles CTAs.
// A row attends keys j < n_cache[row] of its sequence's cache and, under tree attention, the
// provisional slots n_cache + t whose bit t is set in its mask row.  For long contexts with few
// CTAs the keys are also split over S CTAs (chunks [z*C/S, (z+1)*C/S)); then every CTA writes its
// unnormalised (m, l, O) to scratch and the last one to arrive for that (head, row tile) -- found
// with an atomic counter, never by waiting -- merges the splits in split order.
#include "pdl.cuh"
#include "rd_internal.cuh"

namespace rd {

namespace {

constexpr int ROWS = 16;     // rows per CTA (one MMA row tile)
constexpr int KEYS = 64;     // keys per chunk
constexpr int WKEYS = 16;    // keys of a chunk per warp
constexpr int PAD = 8;       // bf16 padding of a shared-memory row (keeps 32-bit and ldmatrix accesses conflict free)
constexpr int MAX_SPLITS = 16;
constexpr int NSTAGE_DEEP = 4;     // K/V chunks in flight per CTA: one CTA per SM (139 KB), the decode-time case
constexpr int NSTAGE_SHALLOW = 2;  // ... three CTAs per SM (70 KB each), for launches of more CTAs than SMs

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int bytes = valid ? 16 : 0;  // zero-fill when the key does not exist
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

#define RD_STAMP(i) asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[i]))

template <int HD, int NSTAGE>
__global__ void __launch_bounds__(128) attention_tc_kernel(const float* __restrict__ qkv,
                                                           const __nv_bfloat16* __restrict__ kc,
                                                           const __nv_bfloat16* __restrict__ vc,
                                                           __nv_bfloat16* __restrict__ out, RowTables rt,
                                                           const int32_t* __restrict__ seq_off, Dims dm, int row_tiles,
                                                           int n_splits, float* __restrict__ scratch,
                                                           int32_t* __restrict__ counters, unsigned long long* dbg, ChainSync cs) {
  unsigned long long t_dbg[6] = {0, 0, 0, 0, 0, 0};
  RD_STAMP(0);
  chain_begin(cs);
#ifdef RD_PROBE_EMPTY_BODIES   // ceiling probe (a build flag, never in the shipped library): keep the hand-off, drop the work
  chain_wait_cta(cs);
  chain_exit(cs);
  return;
#endif
  // Launched inside a chain, the kernel may read before its wait whatever the launches ahead of the chain
  // wrote: the row tables, the tree mask and the cache entries of earlier steps.  Only Q and the K/V of
  // this pass's own rows come from the kernel right before it.
  const bool early = cs.signal_ptr != nullptr;
  if (!early) chain_wait_cta(cs);
  constexpr int LD = HD + PAD;           // shared row stride in bf16
  constexpr int NT = HD / 8;             // output n-tiles
  constexpr int KS = HD / 16;            // k-steps of Q K^T
  constexpr int PW = HD + 4;             // row of a partial: O (unnormalised), m, l, padding (16-byte aligned rows)
  extern __shared__ __align__(16) uint8_t smem[];
  __nv_bfloat16* sKV = reinterpret_cast<__nv_bfloat16*>(smem);                   // [NSTAGE][K | V][KEYS][LD]
  int32_t* s_ncache = reinterpret_cast<int32_t*>(sKV + 2 * NSTAGE * KEYS * LD);  // [ROWS]
  uint32_t* s_mask = reinterpret_cast<uint32_t*>(s_ncache + ROWS);      // [ROWS][MW]
  __shared__ int s_last;

  const int h = blockIdx.x;
  const int b = blockIdx.y / row_tiles, rb = blockIdx.y - b * row_tiles;
  const int z = blockIdx.z;
  const int seq_row0 = seq_off[b], seq_rows = seq_off[b + 1] - seq_row0;
  const int row0 = seq_row0 + rb * ROWS;
  const int nrows = min(ROWS, seq_rows - rb * ROWS);
  if (nrows <= 0) {  // the same for every split and head of this row tile
    if (early) chain_wait_cta(cs);
    chain_exit(cs);
    return;
  }
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
  const int MW = dm.MW;
  const bool tree = rt.mask != nullptr;
  const int r_lo = g, r_hi = g + 8;

  // ---- row tables and mask
  const int nc_seq = rt.n_cache[seq_row0];   // first row of the sequence in this pass
  const int nc_first = rt.n_cache[row0], nc_last = rt.n_cache[row0 + nrows - 1];
  const int nc_mine = (tid < nrows) ? rt.n_cache[row0 + tid] : 0;
  if (tid < ROWS) s_ncache[tid] = nc_mine;
  if (tree) {
    // the mask row of a packed row is its index inside the sequence
    for (int idx = tid; idx < ROWS * MW; idx += 128) {
      const int r = idx / MW, wd = idx - r * MW;
      s_mask[idx] = r < nrows ? rt.mask[((size_t)b * dm.NMAX + rb * ROWS + r) * MW + wd] : 0u;
    }
  }

  // ---- key extent of the tile (the largest key index any of its rows may attend, plus one) and this
  // split's chunk range.  Tree mode: every row of the sequence has the same n_cache and the tree rows
  // follow it.  Causal mode: rows are in position order, the last one reaches furthest.
  const int tree_base = nc_first;
  int kext = tree ? tree_base + seq_rows : nc_last;
  kext = min(kext, dm.max_ctx);
  // keys below this index were written by earlier passes (tree: the context; causal: everything before the
  // slot of the sequence's first row of this pass)
  const int const_keys = tree ? tree_base : nc_seq - 1;
  const int n_chunks = (kext + KEYS - 1) / KEYS;
  const int c_begin = (int)((long long)z * n_chunks / n_splits), c_end = (int)((long long)(z + 1) * n_chunks / n_splits);

  const size_t head_base = ((size_t)b * dm.H + h) * (size_t)dm.max_ctx * HD;
  const uint32_t sKV_u = (uint32_t)__cvta_generic_to_shared(sKV);
  constexpr uint32_t TILE_BYTES = KEYS * LD * 2;
  // asynchronous copy of one chunk's K and V tiles into ring slot `buf` (keys past the extent are
  // zero-filled); always closes a copy group, empty past the last chunk, so the group count is uniform
  // per thread: 16-byte piece c8 of key rows tid/16 + 8j of a chunk (j = 0 .. KEYS/8 - 1 for HD = 128)
  constexpr int PIECES = HD / 8;                 // 16-byte pieces per key row
  constexpr int ROWS_PER_PASS = 128 / PIECES;    // key rows covered by one pass of the 128 threads
  const int cp_row = tid / PIECES, cp_c8 = (tid % PIECES) * 8;
  const __nv_bfloat16* cp_k = kc + head_base + (size_t)cp_row * HD + cp_c8;
  const __nv_bfloat16* cp_v = vc + head_base + (size_t)cp_row * HD + cp_c8;
  const uint32_t cp_dst = sKV_u + (cp_row * LD + cp_c8) * 2;
  auto load_chunk = [&](int ch, int buf) {
    if (ch < c_end) {
      const int k0 = ch * KEYS;
      const uint32_t dk = cp_dst + (2 * buf) * TILE_BYTES, dv = dk + TILE_BYTES;
      if (k0 + KEYS <= kext) {
#pragma unroll
        for (int j = 0; j < KEYS / ROWS_PER_PASS; ++j) {
          const size_t off = (size_t)(k0 + j * ROWS_PER_PASS) * HD;
          cp_async16(dk + j * ROWS_PER_PASS * LD * 2, cp_k + off, true);
          cp_async16(dv + j * ROWS_PER_PASS * LD * 2, cp_v + off, true);
        }
      } else {
#pragma unroll 1
        for (int j = 0; j < KEYS / ROWS_PER_PASS; ++j) {
          const bool valid = k0 + j * ROWS_PER_PASS + cp_row < kext;
          const size_t off = valid ? (size_t)(k0 + j * ROWS_PER_PASS) * HD : (size_t)0;
          cp_async16(dk + j * ROWS_PER_PASS * LD * 2, cp_k + off, valid);
          cp_async16(dv + j * ROWS_PER_PASS * LD * 2, cp_v + off, valid);
        }
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  // the first NSTAGE-1 chunks: those that hold only older keys start before the wait
  int n_pre = 0;
  if (early) {
    while (n_pre < NSTAGE - 1 && (c_begin + n_pre + 1) * KEYS <= const_keys) {
      load_chunk(c_begin + n_pre, n_pre);
      ++n_pre;
    }
    chain_wait_cta(cs);
  }
  RD_STAMP(1);
  // Q of the tile's rows (fp32, rotated by the preceding kernel)
  float2 qraw[KS][4];
  {
    const float* q_lo = qkv + (size_t)(row0 + (r_lo < nrows ? r_lo : 0)) * 3 * dm.d + h * HD + t4 * 2;
    const float* q_hi = qkv + (size_t)(row0 + (r_hi < nrows ? r_hi : 0)) * 3 * dm.d + h * HD + t4 * 2;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qraw[ks][0] = __ldcg(reinterpret_cast<const float2*>(q_lo + ks * 16));
      qraw[ks][1] = __ldcg(reinterpret_cast<const float2*>(q_hi + ks * 16));
      qraw[ks][2] = __ldcg(reinterpret_cast<const float2*>(q_lo + ks * 16 + 8));
      qraw[ks][3] = __ldcg(reinterpret_cast<const float2*>(q_hi + ks * 16 + 8));
    }
  }
  for (int i = n_pre; i < NSTAGE - 1; ++i) load_chunk(c_begin + i, i);

  uint32_t qf[KS][4];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const bool ok = ((e & 1) ? r_hi : r_lo) < nrows;
      qf[ks][e] = ok ? pack_bf16(qraw[ks][e].x, qraw[ks][e].y) : 0u;
    }
  }
  __syncthreads();
  RD_STAMP(2);
  const int nc_lo = s_ncache[r_lo], nc_hi = s_ncache[r_hi];
  const int nc_min = tree ? tree_base : nc_first;   // every valid row of the tile attends at least the keys below this
  const float scale = rsqrtf((float)HD);
  float o[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  for (int ch = c_begin; ch < c_end; ++ch) {
    const int kw = ch * KEYS + warp * WKEYS;   // first key of this warp's share of the chunk
    const int buf = (ch - c_begin) % NSTAGE;
    // chunk ch + NSTAGE - 1 streams into the slot the previous iteration released; then wait until all but
    // the NSTAGE - 1 newest groups have landed, i.e. until chunk ch is in shared memory
    load_chunk(ch + NSTAGE - 1, (ch - c_begin + NSTAGE - 1) % NSTAGE);
    asm volatile("cp.async.wait_group %0;" ::"n"(NSTAGE - 1) : "memory");
    __syncthreads();
    const __nv_bfloat16* sK = sKV + (size_t)(2 * buf) * KEYS * LD + (size_t)warp * WKEYS * LD;
    const uint32_t sV_u = sKV_u + (2 * buf + 1) * TILE_BYTES + warp * WKEYS * LD * 2;

    // ---- S = Q K^T: 16 rows x this warp's 16 keys
    float s[WKEYS / 8][4];
    {
      // two accumulators per key tile (even and odd k-steps): four independent MMA chains instead of two
      float s2[WKEYS / 8][4];
#pragma unroll
      for (int nt = 0; nt < WKEYS / 8; ++nt) {
        s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
        s2[nt][0] = s2[nt][1] = s2[nt][2] = s2[nt][3] = 0.f;
      }
#pragma unroll
      for (int ks = 0; ks < KS; ks += 2) {
#pragma unroll
        for (int nt = 0; nt < WKEYS / 8; ++nt) {
          const __nv_bfloat16* kp = sK + (nt * 8 + g) * LD + t4 * 2;
          const uint32_t b0 = *reinterpret_cast<const uint32_t*>(kp + ks * 16);
          const uint32_t b1 = *reinterpret_cast<const uint32_t*>(kp + ks * 16 + 8);
          const uint32_t b2 = *reinterpret_cast<const uint32_t*>(kp + ks * 16 + 16);
          const uint32_t b3 = *reinterpret_cast<const uint32_t*>(kp + ks * 16 + 24);
          mma_bf16(s[nt], qf[ks], b0, b1);
          mma_bf16(s2[nt], qf[ks + 1], b2, b3);
        }
      }
#pragma unroll
      for (int nt = 0; nt < WKEYS / 8; ++nt) { s[nt][0] += s2[nt][0]; s[nt][1] += s2[nt][1]; s[nt][2] += s2[nt][2]; s[nt][3] += s2[nt][3]; }
    }
    // ---- scale, mask, online softmax (thread holds keys kw + nt*8 + t4*2 + {0,1} of rows r_lo, r_hi)
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
    if (ch * KEYS + KEYS <= nc_min) {
      // every row of the tile attends every key of the chunk
#pragma unroll
      for (int nt = 0; nt < WKEYS / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) s[nt][e] *= scale;
        mx_lo = fmaxf(mx_lo, fmaxf(s[nt][0], s[nt][1]));
        mx_hi = fmaxf(mx_hi, fmaxf(s[nt][2], s[nt][3]));
      }
    } else {
#pragma unroll
      for (int nt = 0; nt < WKEYS / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int key = kw + nt * 8 + t4 * 2 + e;
          bool v_lo = key < nc_lo, v_hi = key < nc_hi;
          if (tree && key >= tree_base) {
            const int tb = key - tree_base;
            if (tb < seq_rows) {
              v_lo = (s_mask[r_lo * MW + (tb >> 5)] >> (tb & 31)) & 1u;
              v_hi = (s_mask[r_hi * MW + (tb >> 5)] >> (tb & 31)) & 1u;
            }
          }
          s[nt][e] = v_lo ? s[nt][e] * scale : -INFINITY;
          s[nt][2 + e] = v_hi ? s[nt][2 + e] * scale : -INFINITY;
          mx_lo = fmaxf(mx_lo, s[nt][e]);
          mx_hi = fmaxf(mx_hi, s[nt][2 + e]);
        }
      }
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float nm_lo = fmaxf(m_lo, mx_lo), nm_hi = fmaxf(m_hi, mx_hi);
    const float corr_lo = (nm_lo == -INFINITY) ? 1.f : __expf(m_lo - nm_lo);
    const float corr_hi = (nm_hi == -INFINITY) ? 1.f : __expf(m_hi - nm_hi);
    const float base_lo = (nm_lo == -INFINITY) ? 0.f : nm_lo, base_hi = (nm_hi == -INFINITY) ? 0.f : nm_hi;
    float sum_lo = 0.f, sum_hi = 0.f;
    uint32_t pf[4];  // P (16 rows x 16 keys) as the A fragment of the P*V product
#pragma unroll
    for (int nt = 0; nt < WKEYS / 8; ++nt) {
      const float p0 = __expf(s[nt][0] - base_lo), p1 = __expf(s[nt][1] - base_lo);
      const float p2 = __expf(s[nt][2] - base_hi), p3 = __expf(s[nt][3] - base_hi);
      sum_lo += p0 + p1;
      sum_hi += p2 + p3;
      pf[nt * 2 + 0] = pack_bf16(p0, p1);
      pf[nt * 2 + 1] = pack_bf16(p2, p3);
    }
    sum_lo += __shfl_xor_sync(0xffffffffu, sum_lo, 1);
    sum_lo += __shfl_xor_sync(0xffffffffu, sum_lo, 2);
    sum_hi += __shfl_xor_sync(0xffffffffu, sum_hi, 1);
    sum_hi += __shfl_xor_sync(0xffffffffu, sum_hi, 2);
    l_lo = l_lo * corr_lo + sum_lo;
    l_hi = l_hi * corr_hi + sum_hi;
    m_lo = nm_lo;
    m_hi = nm_hi;
#pragma unroll
    for (int i = 0; i < NT; ++i) { o[i][0] *= corr_lo; o[i][1] *= corr_lo; o[i][2] *= corr_hi; o[i][3] *= corr_hi; }
    // ---- O += P V : B fragments from this warp's 16 rows of the row-major V tile with ldmatrix.trans
#pragma unroll
    for (int np = 0; np < NT / 2; ++np) {
      uint32_t vb[4];
      const int vrow = (lane & 7) + ((lane >> 3) & 1) * 8;
      const int vcol = np * 16 + (lane >> 4) * 8;
      ldmatrix_x4_trans(vb, sV_u + (vrow * LD + vcol) * 2);
      mma_bf16(o[np * 2], pf, vb[0], vb[1]);
      mma_bf16(o[np * 2 + 1], pf, vb[2], vb[3]);
    }
    __syncthreads();  // every warp is done with this buffer
  }
  RD_STAMP(3);

  // ---- combine the four warps (each saw a quarter of every chunk) through shared memory
  float* s_o = reinterpret_cast<float*>(sKV);          // [4 warps][ROWS][PW]: O, m, l (the K/V tiles are done)
  float* s_w = s_o + 4 * ROWS * PW;                     // [ROWS][MAX_SPLITS] weights of the cross-split merge
  {
    float* mine = s_o + (size_t)warp * ROWS * PW;
#pragma unroll
    for (int i = 0; i < NT; ++i) {
      const int col = i * 8 + t4 * 2;
      *reinterpret_cast<float2*>(mine + r_lo * PW + col) = make_float2(o[i][0], o[i][1]);
      *reinterpret_cast<float2*>(mine + r_hi * PW + col) = make_float2(o[i][2], o[i][3]);
    }
    if (t4 == 0) {
      mine[r_lo * PW + HD] = m_lo; mine[r_lo * PW + HD + 1] = l_lo;
      mine[r_hi * PW + HD] = m_hi; mine[r_hi * PW + HD + 1] = l_hi;
    }
  }
  __syncthreads();
  const int blk = blockIdx.y * gridDim.x + h;  // (sequence, row tile, head)
  float* part = scratch + ((size_t)blk * n_splits + z) * ROWS * PW;   // only touched when n_splits > 1
  for (int idx = tid; idx < ROWS * (HD / 4); idx += 128) {
    const int r = idx / (HD / 4), c = (idx - r * (HD / 4)) * 4;
    float mw[4], gm = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) { mw[w] = s_o[((size_t)w * ROWS + r) * PW + HD]; gm = fmaxf(gm, mw[w]); }
    float L = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float wgt = (mw[w] == -INFINITY) ? 0.f : __expf(mw[w] - gm);
      L += s_o[((size_t)w * ROWS + r) * PW + HD + 1] * wgt;
      const float4 ov = *reinterpret_cast<const float4*>(s_o + ((size_t)w * ROWS + r) * PW + c);
      acc.x += ov.x * wgt; acc.y += ov.y * wgt; acc.z += ov.z * wgt; acc.w += ov.w * wgt;
    }
    if (n_splits == 1) {
      if (r < nrows) {
        const float inv = L > 0.f ? 1.f / L : 0.f;
        *reinterpret_cast<uint2*>(out + (size_t)(row0 + r) * dm.d + h * HD + c) =
            make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
      }
    } else {
      *reinterpret_cast<float4*>(part + r * PW + c) = acc;
      if (c == 0) { part[r * PW + HD] = gm; part[r * PW + HD + 1] = L; }
    }
  }
  RD_STAMP(4);
  if (n_splits == 1) {
    if (dbg && tid == 0) { if (blk == 0) { for (int i = 0; i < 5; ++i) dbg[i] = t_dbg[i]; } atomicMax(dbg + 6, t_dbg[4]); }
    chain_exit(cs);
    return;
  }

  // ---- keys split over CTAs: publish the partial, the last arriver merges the splits in split order
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int old = atomicAdd(counters + blk, 1);
    s_last = (old == n_splits - 1) ? 1 : 0;
    if (old == n_splits - 1) counters[blk] = 0;  // ready for the next launch
  }
  __syncthreads();
  if (dbg && tid == 0 && blk == 0 && z == 0) { for (int i = 0; i < 5; ++i) dbg[i] = t_dbg[i]; }
  if (!s_last) {
    chain_exit(cs);
    return;
  }
  __threadfence();
  const float* all = scratch + (size_t)blk * n_splits * ROWS * PW;
  if (tid < nrows) {
    const int r = tid;
    float mz[MAX_SPLITS], lz[MAX_SPLITS], gm = -INFINITY;
#pragma unroll
    for (int zz = 0; zz < MAX_SPLITS; ++zz) {
      mz[zz] = zz < n_splits ? __ldcg(all + ((size_t)zz * ROWS + r) * PW + HD) : -INFINITY;
      lz[zz] = zz < n_splits ? __ldcg(all + ((size_t)zz * ROWS + r) * PW + HD + 1) : 0.f;
    }
#pragma unroll
    for (int zz = 0; zz < MAX_SPLITS; ++zz) gm = fmaxf(gm, mz[zz]);
    float L = 0.f;
#pragma unroll
    for (int zz = 0; zz < MAX_SPLITS; ++zz) {
      const float wgt = (mz[zz] == -INFINITY) ? 0.f : __expf(mz[zz] - gm);
      L += lz[zz] * wgt;
      mz[zz] = wgt;
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
    for (int zz = 0; zz < MAX_SPLITS; ++zz) s_w[r * MAX_SPLITS + zz] = mz[zz] * inv;
  }
  __syncthreads();
  for (int idx = tid; idx < nrows * (HD / 4); idx += 128) {
    const int r = idx / (HD / 4), c = (idx - r * (HD / 4)) * 4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int z0 = 0; z0 < n_splits; z0 += 4) {
      float4 ov[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        ov[u] = (z0 + u < n_splits) ? __ldcg(reinterpret_cast<const float4*>(all + ((size_t)(z0 + u) * ROWS + r) * PW + c))
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float wgt = (z0 + u < n_splits) ? s_w[r * MAX_SPLITS + z0 + u] : 0.f;
        acc.x += ov[u].x * wgt; acc.y += ov[u].y * wgt; acc.z += ov[u].z * wgt; acc.w += ov[u].w * wgt;
      }
    }
    *reinterpret_cast<uint2*>(out + (size_t)(row0 + r) * dm.d + h * HD + c) =
        make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
  }
  if (dbg && tid == 0 && blk == 0) { RD_STAMP(5); atomicMax(dbg + 6, t_dbg[5]); }
  chain_exit(cs);
}

template <int HD, int NSTAGE>
size_t smem_bytes(int MW) {
  size_t ring = (size_t)(2 * NSTAGE * KEYS) * (HD + PAD) * 2;
  const size_t merge = (size_t)(4 * ROWS * (HD + 4) + ROWS * MAX_SPLITS) * 4;   // the warps' partials reuse the ring
  if (ring < merge) ring = merge;
  return ring + ROWS * 4 + (size_t)ROWS * MW * 4;
}

}  // namespace

size_t attn_tc_scratch_floats(int blocks, int n_splits, int hd) { return (size_t)blocks * n_splits * ROWS * (hd + 4); }
int attn_tc_rows_per_block() { return ROWS; }

cudaError_t attn_tc_prepare(int hd, int MW) {
  cudaError_t e = cudaErrorInvalidValue;
  if (hd == 128) {
    e = cudaFuncSetAttribute(attention_tc_kernel<128, NSTAGE_DEEP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes<128, NSTAGE_DEEP>(MW));
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(attention_tc_kernel<128, NSTAGE_SHALLOW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes<128, NSTAGE_SHALLOW>(MW));
  } else if (hd == 64) {
    e = cudaFuncSetAttribute(attention_tc_kernel<64, NSTAGE_DEEP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes<64, NSTAGE_DEEP>(MW));
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(attention_tc_kernel<64, NSTAGE_SHALLOW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes<64, NSTAGE_SHALLOW>(MW));
  }
  return e;
}

// grid (H, sequences * row_tiles, n_splits); `shallow`: more CTAs than SMs, so several should share an SM
cudaError_t launch_attention_tc(const float* qkv, const void* kcache, const void* vcache, void* out, const RowTables& rt,
                                const int32_t* seq_off, const Dims& dm, int n_seq, int row_tiles, int n_splits,
                                float* scratch, int32_t* counters, unsigned long long* dbg, Chain* chain, int shallow, cudaStream_t st) {
  dim3 grid(dm.H, n_seq * row_tiles, n_splits);
  const ChainSync cs = chain ? chain->link(grid.x * grid.y * grid.z) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
#define RD_ATT_LAUNCH(HD, NST)                                                                                              \
  launch_pdl(attention_tc_kernel<HD, NST>, grid, 128, smem_bytes<HD, NST>(dm.MW), st, qkv, (const __nv_bfloat16*)kcache,    \
             (const __nv_bfloat16*)vcache, (__nv_bfloat16*)out, rt, seq_off, dm, row_tiles, n_splits, scratch, counters, dbg, cs)
  if (dm.hd == 128) {
    if (shallow) RD_ATT_LAUNCH(128, NSTAGE_SHALLOW); else RD_ATT_LAUNCH(128, NSTAGE_DEEP);
  } else if (dm.hd == 64) {
    if (shallow) RD_ATT_LAUNCH(64, NSTAGE_SHALLOW); else RD_ATT_LAUNCH(64, NSTAGE_DEEP);
  } else {
    return cudaErrorInvalidValue;
  }
#undef RD_ATT_LAUNCH
  return cudaGetLastError();
}

}  // namespace rd

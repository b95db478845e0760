// Tree-masked attention for the bf16 path (Sections 3.3, 3.4): KV tiles staged through shared
// memory with 128-bit asynchronous copies, scores and P*V on the tensor cores (mma.sync m16n8k16,
// the work per tile is far too small for tcgen05), online softmax in fp32, split over the keys.
//
// One CTA = (head, sequence, block of up to 64 of its rows, key split).  Each of the 4 warps owns
// 16 rows.  A row attends keys j < n_cache[row] of its sequence's cache and, under tree attention,
// the provisional slots n_cache + t whose bit t is set in its mask row; the split covers the 64-key
// chunks [z*C/S, (z+1)*C/S) of the block's key extent.  With S > 1 every CTA writes its
// unnormalised (m, l, O) to scratch and the last one to arrive for that (head, row block) -- found
// with an atomic counter, never by waiting -- merges the splits in split order and writes the output.
#include "rd_internal.cuh"
#include "pdl.cuh"

namespace rd {

namespace {

constexpr int ROWS = 64;     // rows per CTA (4 warps x 16)
constexpr int KEYS = 64;     // keys per chunk
constexpr int PAD = 8;       // bf16 padding of a shared-memory row (keeps 32-bit and ldmatrix accesses conflict free)

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

template <int HD>
__global__ void __launch_bounds__(128) attention_tc_kernel(const float* __restrict__ qkv,
                                                           const __nv_bfloat16* __restrict__ kc,
                                                           const __nv_bfloat16* __restrict__ vc,
                                                           __nv_bfloat16* __restrict__ out, RowTables rt,
                                                           const int32_t* __restrict__ seq_off, Dims dm, int row_blocks,
                                                           int n_splits, float* __restrict__ scratch,
                                                           int32_t* __restrict__ counters, unsigned long long* dbg) {
  unsigned long long t_dbg[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#define RD_STAMP(i) asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_dbg[i]))
#define RD_DUMP() do { if (dbg && threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0) { \
    if (blockIdx.z == 0) { for (int i_ = 0; i_ < 5; ++i_) dbg[i_] = t_dbg[i_]; } \
    if (t_dbg[5]) atomicMax(dbg + 6, t_dbg[5]); } } while (0)
  RD_STAMP(0);
  pdl_enter();
  RD_STAMP(1);
  constexpr int LD = HD + PAD;           // shared row stride in bf16
  constexpr int NT = HD / 8;             // output n-tiles per warp
  constexpr int KS = HD / 16;            // k-steps of Q K^T
  extern __shared__ __align__(16) uint8_t smem[];
  __nv_bfloat16* sKV = reinterpret_cast<__nv_bfloat16*>(smem);          // [2 buffers][K | V][KEYS][LD]
  int32_t* s_ncache = reinterpret_cast<int32_t*>(sKV + 4 * KEYS * LD);  // [ROWS]
  uint32_t* s_mask = reinterpret_cast<uint32_t*>(s_ncache + ROWS);  // [ROWS][MW]
  __shared__ int s_last;

  const int h = blockIdx.x;
  const int b = blockIdx.y / row_blocks, rb = blockIdx.y - b * row_blocks;
  const int z = blockIdx.z;
  const int seq_row0 = seq_off[b], seq_rows = seq_off[b + 1] - seq_row0;
  const int row0 = seq_row0 + rb * ROWS;
  const int nrows = min(ROWS, seq_rows - rb * ROWS);
  if (nrows <= 0) return;  // the same for every split and head of this row block
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
  const int MW = dm.MW;
  const bool tree = rt.mask != nullptr;

  // ---- key extent of the block (the largest key index any of its rows may attend, plus one) and this
  // split's chunk range.  Tree mode: every row of the sequence has the same n_cache and the tree rows
  // follow it.  Causal mode: rows are in position order, the last one reaches furthest.
  const int tree_base = rt.n_cache[row0];
  int kext = tree ? tree_base + seq_rows : rt.n_cache[row0 + nrows - 1];
  kext = min(kext, dm.max_ctx);
  const int n_chunks = (kext + KEYS - 1) / KEYS;
  const int c_begin = (int)((long long)z * n_chunks / n_splits), c_end = (int)((long long)(z + 1) * n_chunks / n_splits);

  const size_t head_base = ((size_t)b * dm.H + h) * (size_t)dm.max_ctx * HD;
  const uint32_t sKV_u = (uint32_t)__cvta_generic_to_shared(sKV);
  constexpr uint32_t TILE_BYTES = KEYS * LD * 2;
  // asynchronous copy of one chunk's K and V tiles into buffer `buf` (keys past the extent are zero-filled)
  auto load_chunk = [&](int ch, int buf) {
    const int k0 = ch * KEYS;
    for (int idx = tid; idx < KEYS * (HD / 8); idx += 128) {
      const int kr = idx / (HD / 8), c8 = (idx - kr * (HD / 8)) * 8;
      const int key = k0 + kr;
      const bool valid = key < kext;
      const size_t off = head_base + (size_t)(valid ? key : 0) * HD + c8;
      cp_async16(sKV_u + (2 * buf) * TILE_BYTES + (kr * LD + c8) * 2, kc + off, valid);
      cp_async16(sKV_u + (2 * buf + 1) * TILE_BYTES + (kr * LD + c8) * 2, vc + off, valid);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  if (c_begin < c_end) load_chunk(c_begin, 0);   // in flight while Q and the masks are fetched

  // ---- this warp's Q fragments (rows warp*16 + g, +8) straight from global memory into registers: 32
  // independent 8-byte loads per thread, one round trip
  const int r_lo = warp * 16 + g, r_hi = r_lo + 8;
  uint32_t qf[KS][4];
  {
    const float* q_lo = qkv + (size_t)(row0 + (r_lo < nrows ? r_lo : 0)) * 3 * dm.d + h * HD + t4 * 2;
    const float* q_hi = qkv + (size_t)(row0 + (r_hi < nrows ? r_hi : 0)) * 3 * dm.d + h * HD + t4 * 2;
    float2 a[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      a[ks][0] = *reinterpret_cast<const float2*>(q_lo + ks * 16);
      a[ks][1] = *reinterpret_cast<const float2*>(q_hi + ks * 16);
      a[ks][2] = *reinterpret_cast<const float2*>(q_lo + ks * 16 + 8);
      a[ks][3] = *reinterpret_cast<const float2*>(q_hi + ks * 16 + 8);
    }
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool ok = ((e & 1) ? r_hi : r_lo) < nrows;
        qf[ks][e] = ok ? pack_bf16(a[ks][e].x, a[ks][e].y) : 0u;
      }
    }
  }
  for (int r = tid; r < ROWS; r += 128) s_ncache[r] = r < nrows ? rt.n_cache[row0 + r] : 0;
  if (tree) {
    for (int idx = tid; idx < ROWS * MW; idx += 128) {
      const int r = idx / MW, wd = idx - r * MW;
      s_mask[idx] = r < nrows ? rt.mask[((size_t)b * dm.NMAX + rt.local[row0 + r]) * MW + wd] : 0u;
    }
  }
  __syncthreads();
  RD_STAMP(2);
  const int nc_lo = s_ncache[r_lo], nc_hi = s_ncache[r_hi];
  const float scale = rsqrtf((float)HD);
  float o[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  for (int ch = c_begin; ch < c_end; ++ch) {
    const int k0 = ch * KEYS;
    const int buf = (ch - c_begin) & 1;
    // the next chunk streams in while this one is used (its buffer was released by the barrier that
    // ended the previous iteration)
    if (ch + 1 < c_end) {
      load_chunk(ch + 1, buf ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const __nv_bfloat16* sK = sKV + (size_t)(2 * buf) * KEYS * LD;
    const uint32_t sV_u = sKV_u + (2 * buf + 1) * TILE_BYTES;

    // ---- S = Q K^T for this warp's 16 rows x 64 keys
    float s[KEYS / 8][4];
#pragma unroll
    for (int nt = 0; nt < KEYS / 8; ++nt) {
      s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
      const __nv_bfloat16* kp = sK + (nt * 8 + g) * LD + t4 * 2;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(kp + ks * 16);
        const uint32_t b1 = *reinterpret_cast<const uint32_t*>(kp + ks * 16 + 8);
        mma_bf16(s[nt], qf[ks], b0, b1);
      }
    }
    // ---- scale, mask, online softmax (thread holds keys k0 + nt*8 + t4*2 + {0,1} of rows r_lo, r_hi)
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < KEYS / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int key = k0 + nt * 8 + t4 * 2 + e;
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
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float nm_lo = fmaxf(m_lo, mx_lo), nm_hi = fmaxf(m_hi, mx_hi);
    const float corr_lo = (nm_lo == -INFINITY) ? 1.f : __expf(m_lo - nm_lo);
    const float corr_hi = (nm_hi == -INFINITY) ? 1.f : __expf(m_hi - nm_hi);
    const float base_lo = (nm_lo == -INFINITY) ? 0.f : nm_lo, base_hi = (nm_hi == -INFINITY) ? 0.f : nm_hi;
    float sum_lo = 0.f, sum_hi = 0.f;
    uint32_t pf[KEYS / 16][4];  // P as A fragments of the P*V product
#pragma unroll
    for (int nt = 0; nt < KEYS / 8; ++nt) {
      const float p0 = __expf(s[nt][0] - base_lo), p1 = __expf(s[nt][1] - base_lo);
      const float p2 = __expf(s[nt][2] - base_hi), p3 = __expf(s[nt][3] - base_hi);
      sum_lo += p0 + p1;
      sum_hi += p2 + p3;
      pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
      pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
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
    // ---- O += P V : B fragments from the row-major V tile with ldmatrix.trans
#pragma unroll
    for (int kk = 0; kk < KEYS / 16; ++kk) {
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        uint32_t vb[4];
        const int vrow = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int vcol = np * 16 + (lane >> 4) * 8;
        ldmatrix_x4_trans(vb, sV_u + (vrow * LD + vcol) * 2);
        mma_bf16(o[np * 2], pf[kk], vb[0], vb[1]);
        mma_bf16(o[np * 2 + 1], pf[kk], vb[2], vb[3]);
      }
    }
    __syncthreads();  // every warp is done with this buffer
  }

  RD_STAMP(3);
  // ---- results
  if (n_splits == 1) {
    const float inv_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, inv_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
#pragma unroll
    for (int i = 0; i < NT; ++i) {
      const int col = h * HD + i * 8 + t4 * 2;
      if (r_lo < nrows) *reinterpret_cast<uint32_t*>(out + (size_t)(row0 + r_lo) * dm.d + col) = pack_bf16(o[i][0] * inv_lo, o[i][1] * inv_lo);
      if (r_hi < nrows) *reinterpret_cast<uint32_t*>(out + (size_t)(row0 + r_hi) * dm.d + col) = pack_bf16(o[i][2] * inv_hi, o[i][3] * inv_hi);
    }
    return;
  }
  // partial of this split: [ROWS][PW] floats
  constexpr int PW = HD + 4;  // O (unnormalised), m, l, padding to keep rows 16-byte aligned
  const int blk = (blockIdx.y * gridDim.x + h);  // (sequence, row block, head)
  float* mine = scratch + ((size_t)blk * n_splits + z) * ROWS * PW;
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
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int old = atomicAdd(counters + blk, 1);
    s_last = (old == n_splits - 1) ? 1 : 0;
    if (old == n_splits - 1) counters[blk] = 0;  // ready for the next launch
  }
  __syncthreads();
  RD_STAMP(4);
  if (!s_last) { RD_DUMP(); return; }
  __threadfence();
  // ---- merge of the splits, in split order.  Weights of every (row, split) first (into the shared
  // memory the K tile no longer needs), then each thread folds four columns of a row with all its
  // loads in flight at once.
  const float* all = scratch + (size_t)blk * n_splits * ROWS * PW;
  float* s_w = reinterpret_cast<float*>(sKV);           // [ROWS][MAX_SPLITS] weight / L of the row
  constexpr int MAX_SPLITS = 16;
  for (int r = tid; r < nrows; r += 128) {
    float gm = -INFINITY;
    float mz[MAX_SPLITS], lz[MAX_SPLITS];
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
  // four items per thread and iteration, every load of the iteration in flight together
  const int n_items = nrows * (HD / 4);
  for (int base_idx = tid; base_idx < n_items; base_idx += 128 * 4) {
    float4 acc[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int zz = 0; zz < n_splits; ++zz) {
      float4 ov[4];
      float wgt[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int idx = base_idx + u * 128;
        const int r = idx < n_items ? idx / (HD / 4) : 0, c = idx < n_items ? (idx - r * (HD / 4)) * 4 : 0;
        ov[u] = __ldcg(reinterpret_cast<const float4*>(all + ((size_t)zz * ROWS + r) * PW + c));
        wgt[u] = s_w[r * MAX_SPLITS + zz];
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        acc[u].x += ov[u].x * wgt[u]; acc[u].y += ov[u].y * wgt[u]; acc[u].z += ov[u].z * wgt[u]; acc[u].w += ov[u].w * wgt[u];
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int idx = base_idx + u * 128;
      if (idx < n_items) {
        const int r = idx / (HD / 4), c = (idx - r * (HD / 4)) * 4;
        uint2 packed = make_uint2(pack_bf16(acc[u].x, acc[u].y), pack_bf16(acc[u].z, acc[u].w));
        *reinterpret_cast<uint2*>(out + (size_t)(row0 + r) * dm.d + h * HD + c) = packed;
      }
    }
  }
  RD_STAMP(5);
  RD_DUMP();
}

template <int HD>
size_t smem_bytes(int MW) {
  return (size_t)(4 * KEYS) * (HD + PAD) * 2 + ROWS * 4 + (size_t)ROWS * MW * 4;
}

}  // namespace

size_t attn_tc_scratch_floats(int blocks, int n_splits, int hd) { return (size_t)blocks * n_splits * ROWS * (hd + 4); }
int attn_tc_rows_per_block() { return ROWS; }

cudaError_t attn_tc_prepare(int hd, int MW) {
  if (hd == 128)
    return cudaFuncSetAttribute(attention_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes<128>(MW));
  if (hd == 64)
    return cudaFuncSetAttribute(attention_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes<64>(MW));
  return cudaErrorInvalidValue;
}

// grid (H, sequences * row_blocks, n_splits)
cudaError_t launch_attention_tc(const float* qkv, const void* kcache, const void* vcache, void* out, const RowTables& rt,
                                const int32_t* seq_off, const Dims& dm, int n_seq, int row_blocks, int n_splits,
                                float* scratch, int32_t* counters, unsigned long long* dbg, cudaStream_t st) {
  dim3 grid(dm.H, n_seq * row_blocks, n_splits);
  if (dm.hd == 128)
    launch_pdl(attention_tc_kernel<128>, grid, 128, smem_bytes<128>(dm.MW), st, 
        qkv, (const __nv_bfloat16*)kcache, (const __nv_bfloat16*)vcache, (__nv_bfloat16*)out, rt, seq_off, dm, row_blocks,
        n_splits, scratch, counters, dbg);
  else if (dm.hd == 64)
    launch_pdl(attention_tc_kernel<64>, grid, 128, smem_bytes<64>(dm.MW), st, 
        qkv, (const __nv_bfloat16*)kcache, (const __nv_bfloat16*)vcache, (__nv_bfloat16*)out, rt, seq_off, dm, row_blocks,
        n_splits, scratch, counters, dbg);
  else
    return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace rd

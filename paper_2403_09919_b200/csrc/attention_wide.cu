// Tree-masked attention for launches with many rows per sequence (Sections 3.3, 3.4): prompt processing, wide
// beams, large batches.  Same arithmetic as the decode-time kernel -- bf16 operands, scores and P*V on the tensor
// cores (mma.sync m16n8k16), online softmax in fp32 -- but tiled the other way round: one CTA = (head, sequence,
// tile of 64 of its rows); each of the four warps owns 16 rows and walks every key itself, so nothing is merged
// at the end, and a K/V chunk staged in shared memory serves four times as many rows.  With two chunks in flight
// a CTA needs 70 KB, so three are resident per SM where the decode-time kernel, tuned for a handful of row tiles
// with a deep ring, has one.
#include "pdl.cuh"
#include "rd_internal.cuh"

namespace rd {

namespace {

constexpr int WROWS = 64;    // rows per CTA
constexpr int KEYS = 64;     // keys per chunk
constexpr int PAD = 8;       // bf16 padding of a shared-memory row (keeps 32-bit and ldmatrix accesses conflict free)
constexpr int NSTAGE = 3;    // K/V chunks in flight per CTA

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
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
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
__global__ void __launch_bounds__(128, 2) attention_wide_kernel(const float* __restrict__ qkv,
                                                             const __nv_bfloat16* __restrict__ kc,
                                                             const __nv_bfloat16* __restrict__ vc,
                                                             __nv_bfloat16* __restrict__ out, RowTables rt,
                                                             const int32_t* __restrict__ seq_off, Dims dm, int row_tiles,
                                                             ChainSync cs) {
  chain_begin(cs);
  // Launched inside a chain, the kernel may read before its wait whatever the launches ahead of the chain wrote:
  // the row tables and the tree mask.  Q and the K/V of this pass's own rows come from the kernel right before it.
  const bool early = cs.signal_ptr != nullptr;
  if (!early) chain_wait_cta(cs);
  constexpr int LD = HD + PAD;           // shared row stride in bf16
  constexpr int NT = HD / 8;             // output n-tiles
  constexpr int KS = HD / 16;            // k-steps of Q K^T
  extern __shared__ __align__(16) uint8_t smem[];
  __nv_bfloat16* sKV = reinterpret_cast<__nv_bfloat16*>(smem);                   // [NSTAGE][K | V][KEYS][LD]
  int32_t* s_ncache = reinterpret_cast<int32_t*>(sKV + 2 * NSTAGE * KEYS * LD);  // [WROWS]
  uint32_t* s_mask = reinterpret_cast<uint32_t*>(s_ncache + WROWS);              // [WROWS][MW]

  const int h = blockIdx.x;
  const int b = blockIdx.y / row_tiles, rb = blockIdx.y - b * row_tiles;
  const int seq_row0 = seq_off[b], seq_rows = seq_off[b + 1] - seq_row0;
  const int row0 = seq_row0 + rb * WROWS;
  const int nrows = min(WROWS, seq_rows - rb * WROWS);
  if (nrows <= 0) {  // the same for every head of this row tile
    if (early) chain_wait_cta(cs);
    chain_exit(cs);
    return;
  }
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
  const int MW = dm.MW;
  const bool tree = rt.mask != nullptr;
  const int r_lo = warp * 16 + g, r_hi = r_lo + 8;   // this thread's rows inside the tile

  // ---- row tables and mask
  const int nc_first = rt.n_cache[row0], nc_last = rt.n_cache[row0 + nrows - 1];
  if (tid < WROWS) s_ncache[tid] = (tid < nrows) ? rt.n_cache[row0 + tid] : 0;
  if (tree) {
    // the mask row of a packed row is its index inside the sequence
    for (int idx = tid; idx < WROWS * MW; idx += 128) {
      const int r = idx / MW, wd = idx - r * MW;
      s_mask[idx] = r < nrows ? rt.mask[((size_t)b * dm.NMAX + rb * WROWS + r) * MW + wd] : 0u;
    }
  }
  // ---- key extent of the tile (the largest key index any of its rows may attend, plus one).  Tree mode: every
  // row of the sequence has the same n_cache and the tree rows follow it.  Causal mode: rows are in position
  // order, the last one reaches furthest.
  const int tree_base = nc_first;
  int kext = tree ? tree_base + seq_rows : nc_last;
  kext = min(kext, dm.max_ctx);
  const int n_chunks = (kext + KEYS - 1) / KEYS;
  // the keys this warp's rows can reach (causal mode: a warp whose rows come early stops early)
  int wext = kext;
  if (!tree) wext = (warp * 16 < nrows) ? min(kext, rt.n_cache[row0 + min(warp * 16 + 15, nrows - 1)]) : 0;
  if (warp * 16 >= nrows) wext = 0;

  const size_t head_base = ((size_t)b * dm.H + h) * (size_t)dm.max_ctx * HD;
  const uint32_t sKV_u = (uint32_t)__cvta_generic_to_shared(sKV);
  constexpr uint32_t TILE_BYTES = KEYS * LD * 2;
  constexpr int PIECES = HD / 8;                 // 16-byte pieces per key row
  constexpr int ROWS_PER_PASS = 128 / PIECES;    // key rows covered by one pass of the 128 threads
  const int cp_row = tid / PIECES, cp_c8 = (tid % PIECES) * 8;
  const __nv_bfloat16* cp_k = kc + head_base + (size_t)cp_row * HD + cp_c8;
  const __nv_bfloat16* cp_v = vc + head_base + (size_t)cp_row * HD + cp_c8;
  const uint32_t cp_dst = sKV_u + (cp_row * LD + cp_c8) * 2;
  // asynchronous copy of one chunk's K and V tiles into ring slot `buf` (keys past the extent are zero-filled);
  // always closes a copy group, empty past the last chunk, so the group count is uniform
  auto load_chunk = [&](int ch, int buf) {
    if (ch < n_chunks) {
      const int k0 = ch * KEYS;
      const uint32_t dk = cp_dst + (2 * buf) * TILE_BYTES, dv = dk + TILE_BYTES;
      const bool whole = k0 + KEYS <= kext;
#pragma unroll
      for (int j = 0; j < KEYS / ROWS_PER_PASS; ++j) {
        const bool valid = whole || (k0 + j * ROWS_PER_PASS + cp_row < kext);
        const size_t off = valid ? (size_t)(k0 + j * ROWS_PER_PASS) * HD : (size_t)0;
        cp_async16(dk + j * ROWS_PER_PASS * LD * 2, cp_k + off, valid);
        cp_async16(dv + j * ROWS_PER_PASS * LD * 2, cp_v + off, valid);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  if (early) chain_wait_cta(cs);
#pragma unroll
  for (int i = 0; i < NSTAGE - 1; ++i) load_chunk(i, i);

  // Q of this warp's rows (fp32, rotated by the preceding kernel) as bf16 A fragments
  uint32_t qf[KS][4];
  {
    const bool ok_lo = r_lo < nrows, ok_hi = r_hi < nrows;
    const float* q_lo = qkv + (size_t)(row0 + (ok_lo ? r_lo : 0)) * 3 * dm.d + h * HD + t4 * 2;
    const float* q_hi = qkv + (size_t)(row0 + (ok_hi ? r_hi : 0)) * 3 * dm.d + h * HD + t4 * 2;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const float2 a = __ldcg(reinterpret_cast<const float2*>(q_lo + ks * 16));
      const float2 bq = __ldcg(reinterpret_cast<const float2*>(q_hi + ks * 16));
      const float2 c = __ldcg(reinterpret_cast<const float2*>(q_lo + ks * 16 + 8));
      const float2 e = __ldcg(reinterpret_cast<const float2*>(q_hi + ks * 16 + 8));
      qf[ks][0] = ok_lo ? pack_bf16(a.x, a.y) : 0u;
      qf[ks][1] = ok_hi ? pack_bf16(bq.x, bq.y) : 0u;
      qf[ks][2] = ok_lo ? pack_bf16(c.x, c.y) : 0u;
      qf[ks][3] = ok_hi ? pack_bf16(e.x, e.y) : 0u;
    }
  }
  __syncthreads();   // row tables and mask are in shared memory
  const int nc_lo = s_ncache[r_lo], nc_hi = s_ncache[r_hi];
  const int nc_min = tree ? tree_base : nc_first;   // every valid row of the tile attends at least the keys below this
  const float scale = rsqrtf((float)HD);
  float o[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  for (int ch = 0; ch < n_chunks; ++ch) {
    const int k0 = ch * KEYS;
    const int buf = ch % NSTAGE;
    load_chunk(ch + NSTAGE - 1, (ch + NSTAGE - 1) % NSTAGE);   // into the slot the previous iteration released
    asm volatile("cp.async.wait_group %0;" ::"n"(NSTAGE - 1) : "memory");
    __syncthreads();
    if (k0 < wext) {
      const uint32_t sK_u = sKV_u + (2 * buf) * TILE_BYTES;
      const uint32_t sV_u = sK_u + TILE_BYTES;
      // ---- S = Q K^T: 16 rows x 64 keys.  One ldmatrix.x4 fetches the B fragments of two k-steps of a key tile.
      float s[KEYS / 8][4];
#pragma unroll
      for (int nt = 0; nt < KEYS / 8; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
      for (int ks = 0; ks < KS; ks += 2) {
#pragma unroll
        for (int nt = 0; nt < KEYS / 8; ++nt) {
          uint32_t kb[4];   // matrices: (keys nt*8.., dims ks*16 + {0, 8, 16, 24})
          ldmatrix_x4(kb, sK_u + ((nt * 8 + (lane & 7)) * LD + ks * 16 + (lane >> 3) * 8) * 2);
          mma_bf16(s[nt], qf[ks], kb[0], kb[1]);
          mma_bf16(s[nt], qf[ks + 1], kb[2], kb[3]);
        }
      }
      // ---- scale, mask, online softmax (thread holds keys k0 + nt*8 + t4*2 + {0,1} of rows r_lo, r_hi)
      float mx_lo = -INFINITY, mx_hi = -INFINITY;
      if (k0 + KEYS <= nc_min) {
#pragma unroll
        for (int nt = 0; nt < KEYS / 8; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) s[nt][e] *= scale;
          mx_lo = fmaxf(mx_lo, fmaxf(s[nt][0], s[nt][1]));
          mx_hi = fmaxf(mx_hi, fmaxf(s[nt][2], s[nt][3]));
        }
      } else {
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
      uint32_t pf[KEYS / 16][4];  // P (16 rows x 64 keys) as A fragments of the P*V product
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
    }
    __syncthreads();  // every warp is done with this buffer
  }

  // ---- each warp normalises and writes its own rows
  {
    const float inv_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, inv_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
    __nv_bfloat16* o_lo = out + (size_t)(row0 + r_lo) * dm.d + h * HD + t4 * 2;
    __nv_bfloat16* o_hi = out + (size_t)(row0 + r_hi) * dm.d + h * HD + t4 * 2;
#pragma unroll
    for (int i = 0; i < NT; ++i) {
      if (r_lo < nrows) *reinterpret_cast<uint32_t*>(o_lo + i * 8) = pack_bf16(o[i][0] * inv_lo, o[i][1] * inv_lo);
      if (r_hi < nrows) *reinterpret_cast<uint32_t*>(o_hi + i * 8) = pack_bf16(o[i][2] * inv_hi, o[i][3] * inv_hi);
    }
  }
  chain_exit(cs);
}

template <int HD>
size_t wide_smem_bytes(int MW) {
  return (size_t)(2 * NSTAGE * KEYS) * (HD + PAD) * 2 + WROWS * 4 + (size_t)WROWS * MW * 4;
}

}  // namespace

int attn_wide_rows_per_block() { return WROWS; }

cudaError_t attn_wide_prepare(int hd, int MW) {
  if (hd == 128)
    return cudaFuncSetAttribute(attention_wide_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)wide_smem_bytes<128>(MW));
  if (hd == 64)
    return cudaFuncSetAttribute(attention_wide_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)wide_smem_bytes<64>(MW));
  return cudaErrorInvalidValue;
}

// grid (H, sequences * row_tiles): row_tiles tiles of 64 rows cover the longest sequence of the launch
cudaError_t launch_attention_wide(const float* qkv, const void* kcache, const void* vcache, void* out, const RowTables& rt,
                                  const int32_t* seq_off, const Dims& dm, int n_seq, int row_tiles, Chain* chain, cudaStream_t st) {
  dim3 grid(dm.H, n_seq * row_tiles);
  const ChainSync cs = chain ? chain->link(grid.x * grid.y) : ChainSync{nullptr, 0u, nullptr, nullptr, nullptr};
  if (dm.hd == 128)
    launch_pdl(attention_wide_kernel<128>, grid, 128, wide_smem_bytes<128>(dm.MW), st, qkv, (const __nv_bfloat16*)kcache,
               (const __nv_bfloat16*)vcache, (__nv_bfloat16*)out, rt, seq_off, dm, row_tiles, cs);
  else if (dm.hd == 64)
    launch_pdl(attention_wide_kernel<64>, grid, 128, wide_smem_bytes<64>(dm.MW), st, qkv, (const __nv_bfloat16*)kcache,
               (const __nv_bfloat16*)vcache, (__nv_bfloat16*)out, rt, seq_off, dm, row_tiles, cs);
  else
    return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace rd

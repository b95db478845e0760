// Internal declarations shared by the translation units of libredrafter.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "chain.cuh"
#include "gemm_out.cuh"
#include "redrafter.h"

namespace rd {

// ---- device status word bits (OR-ed by kernels, read by redrafter_poll) ----
enum : int {
  DEV_ERR_TOKEN_RANGE = 1 << 0,  // a token id outside [0, vocab) was clamped
  DEV_ERR_INDEX_RANGE = 1 << 1,  // a packed/unpack/slot index outside its range was skipped
  DEV_ERR_TIMEOUT = 1 << 2,      // a bounded wait (mbarrier) gave up
  DEV_ERR_CAPACITY = 1 << 3      // a KV slot beyond max_ctx was skipped
};

// ---- element type helpers ----
template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float silu_f(float v) { return v / (1.0f + __expf(-v)); }

// Row tables of one forward pass over M rows (device memory).  A row is one token of one
// sequence; it attends cache slots [0, n_cache) of its sequence plus, when mask != nullptr,
// the rows (seq_rowbase[seq] + j) whose bit j is set in its mask row (tree attention).
struct RowTables {
  const int32_t* tok;         // [M] token id
  const int32_t* seq;         // [M] sequence index b
  const int32_t* pos;         // [M] position id (rotary embedding)
  const int32_t* slot;        // [M] cache slot the row's K/V are written to
  const int32_t* n_cache;     // [M] number of leading cache slots the row attends
  const int32_t* local;       // [M] index of the row inside its sequence's group of rows (its mask row)
  const uint32_t* mask;       // [B][NMAX][MW] tree mask or nullptr (causal: n_cache covers everything)
  const int32_t* m_total;     // [1] number of valid rows (device)
};

struct Dims {
  int n_layers, d, H, hd, F, V, dr, dh, n_head_layers;
  int B, max_ctx, BW, L, NMAX, MW;
  float eps, theta;
  int dtype;
};

// ---- launchers (definitions in the .cu files; all enqueue on `st`, return cudaGetLastError) ----
// Y[m][n] = sum_k A[m][k] W[n][k], M rows given by *m_total (<= m_max), on CUDA cores.  Fills *out_desc.
cudaError_t launch_gemm_simt(int dtype, const void* A, int lda, const void* W, int N, int K, const int32_t* m_total,
                             int m_max, float* raw, int ld_raw, GemmOut* out_desc, cudaStream_t st);

// Tensor-core (tcgen05) projection, bf16 only.  Operands are passed as TMA descriptors.
int tc_make_map(void* out_map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows);
int tc_weight_box_rows();
int tc_pick_mt(int m_max);
size_t tc_partial_floats(int grid, int mt);
cudaError_t tc_prepare(int* smem_limit_out, int* pairs_out);
bool tc_use_pairs(int m_max, int N, int grid, int pairs, int min_rows);
double tc_last_prefetch_bytes();
cudaError_t launch_gemm_tc(const void* map_w, const void* const map_a[16], int N, int K, const int32_t* m_total, int m_max,
                           float* raw, int ld_raw, float* partial, int32_t* status, int grid, int pairs, int smem_limit,
                           unsigned long long* trace, GemmOut* out_desc, Chain* chain, int pair, cudaStream_t st);

cudaError_t launch_embed(int dtype, const void* emb, const int32_t* tok, float* x, int d, int V, const int32_t* m_total,
                         int m_max, int* status, cudaStream_t st);
cudaError_t launch_rmsnorm(int dtype, float* x, const GemmOut* proj, const void* gain, void* out_t, float* out_f32, int d,
                           float eps, const int32_t* m_total, int m_max, Chain* chain, cudaStream_t st);
cudaError_t launch_rope_table(const int32_t* pos, float* table, int hd, float theta, const int32_t* m_total, int m_max,
                              cudaStream_t st);
cudaError_t launch_rope_kv(int dtype, float* qkv, const GemmOut& proj, void* kcache, void* vcache, const float* table,
                           const RowTables& rt, const Dims& dm, int m_max, int* status, Chain* chain, cudaStream_t st);
cudaError_t launch_attention(int dtype, const float* qkv, const void* kcache, const void* vcache, void* out_t,
                             const RowTables& rt, const Dims& dm, int m_max, cudaStream_t st);
// Tensor-core attention (bf16): KV tiles staged through shared memory, split over the keys.
size_t attn_tc_scratch_floats(int blocks, int n_splits, int hd);
// many rows per sequence (prompts, wide beams, large batches): tiles of 64 rows, a warp per 16 of them
// head dimension 128, many rows per sequence: tcgen05 attention, tiles of 128 rows
int attn_t5_rows_per_block();
bool attn_t5_supported(int hd);
cudaError_t attn_t5_prepare(int hd, int MW);
cudaError_t launch_attention_t5(const void* map_k, const void* map_v, const float* qkv, void* out, const RowTables& rt,
                                const int32_t* seq_off, const int32_t* seq_order, const Dims& dm, int n_seq, int row_tiles, int32_t* status, Chain* chain,
                                cudaStream_t st);
int attn_wide_rows_per_block();
cudaError_t attn_wide_prepare(int hd, int MW);
cudaError_t launch_attention_wide(const float* qkv, const void* kcache, const void* vcache, void* out, const RowTables& rt,
                                  const int32_t* seq_off, const Dims& dm, int n_seq, int row_tiles, Chain* chain, cudaStream_t st);
int attn_tc_rows_per_block();
cudaError_t attn_tc_prepare(int hd, int MW);
cudaError_t launch_attention_tc(const float* qkv, const void* kcache, const void* vcache, void* out, const RowTables& rt,
                                const int32_t* seq_off, const Dims& dm, int n_seq, int row_blocks, int n_splits,
                                float* scratch, int32_t* counters, unsigned long long* dbg, Chain* chain, int shallow, cudaStream_t st);
cudaError_t elementwise_prepare(int dtype);
cudaError_t drafter_prepare(int dtype);
cudaError_t launch_swiglu(int dtype, const GemmOut& proj, void* out_t, int F, const int32_t* m_total, int m_max,
                          int32_t* status, Chain* chain, cudaStream_t st);
// Token choice at temperature > 0: inv_t = 1 / temperature (0: greedy), (k0, k1) the seed's two halves.
struct Sampling {
  float inv_t;
  uint32_t k0, k1;
};
cudaError_t launch_argmax_rows(float* logits, const GemmOut& proj, int V, int32_t* out, const int32_t* out_index,
                               const int32_t* m_total, int m_max, const Sampling& smp, const int32_t* row_seq,
                               const int32_t* row_pos, int pos_add, cudaStream_t st);

// drafter
cudaError_t launch_draft_init(int dtype, const void* emb, const int32_t* root, const float* h, void* x_t, float* x_f,
                              void* se_t, const Dims& dm, int B, int* status, cudaStream_t st);
cudaError_t launch_act(int dtype, const GemmOut& proj, const void* bias, const float* resid, int ld_resid, float* out_f,
                       void* out_t, int ld_out, int N, const int32_t* m_total, int m_max, Chain* chain, cudaStream_t st);
// Scratch of the two-kernel selection (seg_max == nullptr: single-kernel selection only).
struct SelectScratch {
  float *seg_max, *seg_sum, *seg_val;   // [rows][32], [rows][32], [rows][512]
  int32_t* seg_idx;                     // [rows][512]
  int grid_hint;                        // CTAs to aim for (the SM count)
  unsigned long long* top;              // [rows][BW] keys of every row's BW best continuations
};
int draft_select_segments(const Dims& dm, int rows, int grid_hint);
cudaError_t launch_draft_select(int dtype, const GemmOut& proj, int call, float* lse, float* val, int32_t* idx,
                                const float* score_in, float* score_out, const int32_t* hist_in, int32_t* hist_out,
                                const void* emb, const float* s_new_f, int ld_s, void* se_t, const Dims& dm, int B,
                                int32_t* beams_out, float* scores_out, int32_t* counters, const int32_t* m_total,
                                unsigned long long* dbg, const SelectScratch& sc, Chain* chain, cudaStream_t st);
cudaError_t launch_fill_h(int dtype, const float* h, void* x_t, float* x_f, const Dims& dm, int B, cudaStream_t st);

// pack / accept
cudaError_t launch_pack(const int32_t* beams, const int32_t* root, const int32_t* ctx, const rd_packed& out,
                        const Dims& dm, int B, int no_tree, cudaStream_t st);
cudaError_t launch_build_rows_tree(const rd_packed& pk, const int32_t* ctx, int32_t* row_tok, int32_t* row_seq,
                                   int32_t* row_pos, int32_t* row_slot, int32_t* row_ncache, int32_t* row_local,
                                   int32_t* row_out_index, int32_t* seq_off, int32_t* seq_order, int32_t* m_total, const Dims& dm, int B,
                                   int* status, cudaStream_t st);
cudaError_t launch_build_rows_ar(const int32_t* root, const int32_t* ctx, int32_t* row_tok, int32_t* row_seq,
                                 int32_t* row_pos, int32_t* row_slot, int32_t* row_ncache, int32_t* row_local,
                                 int32_t* row_out_index, int32_t* seq_off, int32_t* m_total, const Dims& dm, int B,
                                 int* status, cudaStream_t st);
cudaError_t launch_scatter_rows(const float* src, int width, float* dst, const int32_t* row_out_index,
                                const int32_t* m_total, int m_max, cudaStream_t st);
cudaError_t launch_cast_rows(int dtype, const float* src, void* dst, int n, cudaStream_t st);
cudaError_t launch_fill_i32(int32_t* p, int32_t v, int n, cudaStream_t st);
cudaError_t launch_accept(int dtype, const int32_t* beams, const rd_packed& pk, const int32_t* argmax,
                          const float* hidden, void* kcache, int32_t* ctx, int32_t* root, float* h,
                          const rd_accept_out& out, int32_t* n_accept_ws, int32_t* best_ws, int32_t* ctx_prev,
                          const Dims& dm, int B, int* status, cudaStream_t st);
int accept_static_max_batch();
cudaError_t accept_static_scratch(int32_t** n_accept, int32_t** best, int32_t** ctx_prev);
cudaError_t launch_ar_finish(const int32_t* argmax_c, const float* hidden_c, int32_t* ctx, int32_t* root, float* h,
                             int32_t* token_out, const Dims& dm, int B, cudaStream_t st);
cudaError_t launch_prefill_finish(const float* hidden_c, const int32_t* last_row, float* h, int d, int B,
                                  cudaStream_t st);

}  // namespace rd

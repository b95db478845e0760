// C-ABI entry points (include/redrafter.h): handle, workspace carve-up, and the host-side
// sequencing of the kernels of one speculative decode step (Section 3.4).  No kernel here.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cmath>
#include <map>
#include <new>
#include <unordered_map>
#include <utility>
#include <vector>

#include "rd_internal.cuh"

using namespace rd;

namespace {

struct Bump {  // carve-up of the caller's workspace; with base == nullptr it only measures
  char* base;
  size_t off;
  template <typename T> T* take(size_t count) {
    off = (off + 255) & ~size_t(255);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

struct Workspace {
  // decode state
  int32_t *ctx, *root, *status;
  float* h;
  // row tables of the current forward
  int32_t *row_tok, *row_seq, *row_pos, *row_slot, *row_ncache, *row_local, *row_out_index, *m_total, *last_row, *seq_off, *seq_order;
  // activations of the forward (compact rows)
  float *x, *qkv, *proj_d, *gu, *hidden_f, *logits, *rope_tab;
  void *a_t, *attn_t, *act_t, *hidden_t, *h_t;
  int32_t* argmax_c;
  // step-internal packed beam, beams, verify outputs, accept scratch
  rd_packed pk;
  int32_t *beams, *argmax_p, *n_accept, *best, *ctx_prev, *acc_tokens;
  float *scores, *hidden_p;
  // drafter
  void *xc_t, *x0_t, *x1_t, *x2_t, *se_t, *uw;   // se_t: [R][d_rnn + d] = [s ; e]; uw: [d_rnn][d_rnn + d] = [U W]
  float *xc_f, *x0_f, *x1_f, *x2_f, *sraw, *hraw, *dlogits, *lse, *cand_val, *score_a, *score_b;
  int32_t *cand_idx, *hist_a, *hist_b, *one_b, *one_r;
  float *seg_max, *seg_sum, *seg_val;   // two-kernel selection: per (row, segment) maximum, sum, candidates
  int32_t* seg_idx;
  unsigned long long* sel_top;          // [rows][BW] keys of every row's BW best continuations
  // tensor-core projection scratch
  float* tc_partial;
  // tensor-core attention scratch
  int32_t *att_counters, *sel_counters;
  unsigned int* chain_ctr;  // counters of the launch-to-launch hand-off
  float* att_scratch;
  unsigned long long* trace;  // [TRACE_SLOTS][8] timestamps of traced projection launches
};

size_t esize(int dtype) { return dtype == RD_DTYPE_FP32 ? 4 : 2; }

struct alignas(64) TensorMapBox {  // opaque storage of one CUtensorMap (128 bytes) + the matrix it describes
  unsigned char bytes[128];
  int rows, cols;
};

}  // namespace

// timing classes of redrafter_profile_read
enum { PROF_GEMM = 0, PROF_ATTN = 1, PROF_NORM = 2, PROF_ROPE = 3, PROF_SWIGLU = 4, PROF_DRAFT_SMALL = 5, PROF_PACK_ACCEPT = 6,
       PROF_MISC = 7, PROF_CLASSES = 8 };

struct rd_handle {
  rd_config cfg;
  Dims dm;
  int m_cap;  // rows one forward pass can hold
  Workspace ws;
  char* kv;
  size_t kv_plane;  // elements per (layer, K|V) plane
  std::vector<const void*> attn_norm, wqkv, wo, ffn_norm, w_gate_up, w_down, head_w, head_b;
  rd_weights w;
  bool prefilled;
  int batch;      // active sequences
  int ctx_bound;  // host-side upper bound of every sequence's context length
  Sampling sampling;  // how the LLM's tokens are chosen (inv_t = 0: greedy)
  int64_t launches;
  int64_t route[RD_ROUTE_COUNT];  // launches per kernel variant (redrafter_route_counts)
  // tensor-core path (bf16): TMA descriptors by base pointer, launch geometry
  bool use_tc;
  int trace_next;  // next trace slot, -1 = tracing off
  std::vector<double> trace_bytes;  // weight bytes of each traced launch (0: not a projection)
  std::vector<double> trace_prefetch;  // ... of which requested before the launch's dependency wait
  int tc_grid, tc_smem;
  const int32_t* att_seq_order = nullptr;   // sequences longest first for the pass being enqueued, or nullptr
  int tc_pairs;   // CTA pairs of the pair projection kernel that fit the device at once (0: not used)
  int tc_pairs_avail, tc_pairs_min_rows;   // the pairs the device offers; row bound from which launches use them
  bool tc_pairs_prefill;
  std::vector<TensorMapBox> kv_maps;   // [layer][K | V]: cache planes as [sequences * heads * max_ctx][head dim] matrices
  Chain chain;  // counter hand-off between the launches of a forward pass
  bool chain_dirty;  // a launch failed after the chain had counted it: reset the counters before the next pass
  int device;        // ordinal of the device the handle was made on
  // Context-bound feedback: after a step the device-side context lengths are copied to pinned host memory without
  // waiting; a later call that finds the copy complete tightens the host-side bound with it.
  int32_t* fb_host;          // [2][max_batch] pinned
  cudaEvent_t fb_event[2];
  bool fb_pending[2];
  int64_t fb_growth_at[2];   // value of fb_growth when the copy was enqueued
  int64_t fb_growth;         // tokens by which a sequence's context can have grown since the handle was made
  int fb_next;
  unsigned fb_calls;         // a copy is enqueued on every eighth call: the bound lags by at most 8 (1 + L) tokens
  std::unordered_map<const void*, TensorMapBox> maps;               // weights
  std::unordered_map<const void*, std::pair<int, int>> act_shape;   // activation buffers: rows, cols
  std::map<std::pair<const void*, int>, TensorMapBox> act_maps;     // by (buffer, rows per box), made on first use
  // optional per-launch timing of the projections (class 0) and the attention kernel (class 1)
  bool profiling;
  std::vector<cudaEvent_t> ev[PROF_CLASSES];   // start/stop pairs
  size_t ev_used[PROF_CLASSES];
  double prof_ms[PROF_CLASSES], prof_bytes[PROF_CLASSES];
  int64_t prof_n[PROF_CLASSES];
  char err[512];
};

namespace {

char g_init_err[512] = "";  // why the last redrafter_init failed (there is no handle to hold it)

int init_fail(rd_handle* h, int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_init_err, sizeof(g_init_err), fmt, ap);
  va_end(ap);
  delete h;
  return code;
}

int fail(rd_handle* h, int code, const char* fmt, ...) {
  if (h && code == RD_ERR_CUDA) h->chain_dirty = true;
  if (h) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(h->err, sizeof(h->err), fmt, ap);
    va_end(ap);
  }
  return code;
}

bool make_dims(const rd_config* c, Dims* dm) {
  if (!c || c->struct_bytes != (int32_t)sizeof(rd_config)) return false;
  if (c->n_layers <= 0 || c->d_model <= 0 || c->n_heads <= 0 || c->d_ffn <= 0 || c->vocab <= 0) return false;
  if (c->d_model % c->n_heads) return false;
  if (c->max_batch <= 0 || c->max_ctx <= 0 || c->beam_width <= 0 || c->beam_length <= 0) return false;
  if (c->dtype != RD_DTYPE_FP32 && c->dtype != RD_DTYPE_BF16) return false;
  if (c->n_head_layers < 0 || c->d_rnn != c->d_model) return false;
  dm->n_layers = c->n_layers; dm->d = c->d_model; dm->H = c->n_heads; dm->hd = c->d_model / c->n_heads;
  dm->F = c->d_ffn; dm->V = c->vocab; dm->dr = c->d_rnn; dm->dh = c->d_rnn + c->d_model;
  dm->n_head_layers = c->n_head_layers; dm->B = c->max_batch; dm->max_ctx = c->max_ctx;
  dm->BW = c->beam_width; dm->L = c->beam_length; dm->NMAX = 1 + c->beam_width * c->beam_length;
  dm->MW = (dm->NMAX + 31) / 32; dm->eps = c->rms_eps; dm->theta = c->rope_theta; dm->dtype = c->dtype;
  return true;
}

int shape_ok(const Dims& dm) {
  const int vec = dm.dtype == RD_DTYPE_FP32 ? 4 : 8;
  if (dm.hd != 64 && dm.hd != 128) return 0;
  if (dm.d % vec || dm.F % vec || dm.dh % vec || dm.V % 4) return 0;
  if (dm.BW > dm.V || dm.BW > 128) return 0;
  if (dm.BW * (dm.L + 1) > 1024 || dm.NMAX > 1024) return 0;
  return 1;
}

constexpr int TRACE_SLOTS = 512;
constexpr int TC_MAX_GRID = 160;  // upper bound of the SM count the scratch is sized for
constexpr int ATT_MAX_SPLIT_BLOCKS = 4 * TC_MAX_GRID;  // (blocks x splits) the split-KV scratch holds

// Rows one forward pass can hold: a verification pass needs B x NMAX; prompt processing takes passes of this many
// rows, and every pass streams all weights, so the floor is four row tiles (the workspace grows by about 0.2 MB per
// row at the 7B shape).
int m_cap_of(const Dims& dm) {
  const int v = dm.B * dm.NMAX;
  return v > 1024 ? v : 1024;
}

void carve(Bump& bp, const Dims& dm, int m_cap, Workspace* w) {
  const size_t es = esize(dm.dtype);
  const int B = dm.B, R = dm.B * dm.BW, C = dm.L + 1;
  w->ctx = bp.take<int32_t>(B); w->root = bp.take<int32_t>(B); w->status = bp.take<int32_t>(4);
  w->h = bp.take<float>((size_t)B * dm.d);
  w->row_tok = bp.take<int32_t>(m_cap); w->row_seq = bp.take<int32_t>(m_cap); w->row_pos = bp.take<int32_t>(m_cap);
  w->row_slot = bp.take<int32_t>(m_cap); w->row_ncache = bp.take<int32_t>(m_cap); w->row_local = bp.take<int32_t>(m_cap);
  w->row_out_index = bp.take<int32_t>(m_cap); w->m_total = bp.take<int32_t>(4); w->last_row = bp.take<int32_t>(B);
  w->one_b = bp.take<int32_t>(4); w->one_r = bp.take<int32_t>(4);
  w->seq_off = bp.take<int32_t>(B + 1);
  w->seq_order = bp.take<int32_t>(B);
  w->att_counters = bp.take<int32_t>(ATT_MAX_SPLIT_BLOCKS);
  w->sel_counters = bp.take<int32_t>(B);
  w->chain_ctr = bp.take<unsigned int>(CHAIN_SLOTS);
  w->x = bp.take<float>((size_t)m_cap * dm.d);
  w->qkv = bp.take<float>((size_t)m_cap * 3 * dm.d);
  w->proj_d = bp.take<float>((size_t)m_cap * dm.d);
  w->gu = bp.take<float>((size_t)m_cap * 2 * dm.F);
  w->hidden_f = bp.take<float>((size_t)m_cap * dm.d);
  w->logits = bp.take<float>((size_t)dm.B * dm.NMAX * dm.V);   // verification rows only (prompt passes need B rows)
  w->rope_tab = bp.take<float>((size_t)m_cap * dm.hd);
  w->a_t = bp.take<char>((size_t)m_cap * dm.d * es);
  w->attn_t = bp.take<char>((size_t)m_cap * dm.d * es);
  w->act_t = bp.take<char>((size_t)m_cap * dm.F * es);
  w->hidden_t = bp.take<char>((size_t)m_cap * dm.d * es);
  w->h_t = bp.take<char>((size_t)B * dm.d * es);
  w->argmax_c = bp.take<int32_t>(m_cap);
  w->pk.tokens = bp.take<int32_t>((size_t)B * dm.NMAX); w->pk.n = bp.take<int32_t>(B);
  w->pk.unpack = bp.take<int32_t>((size_t)R * C); w->pk.pos = bp.take<int32_t>((size_t)B * dm.NMAX);
  w->pk.mask = bp.take<uint32_t>((size_t)B * dm.NMAX * dm.MW); w->pk.parent = bp.take<int32_t>((size_t)B * dm.NMAX);
  w->beams = bp.take<int32_t>((size_t)R * dm.L); w->argmax_p = bp.take<int32_t>((size_t)B * dm.NMAX);
  w->n_accept = bp.take<int32_t>(B); w->best = bp.take<int32_t>(B); w->ctx_prev = bp.take<int32_t>(B);
  w->acc_tokens = bp.take<int32_t>((size_t)B * C);
  w->scores = bp.take<float>(R); w->hidden_p = bp.take<float>((size_t)B * dm.NMAX * dm.d);
  w->xc_t = bp.take<char>((size_t)B * dm.dh * es); w->x0_t = bp.take<char>((size_t)R * dm.dh * es);
  w->x1_t = bp.take<char>((size_t)R * dm.dh * es); w->x2_t = bp.take<char>((size_t)R * dm.dh * es);
  w->se_t = bp.take<char>((size_t)R * (dm.dr + dm.d) * es); w->uw = bp.take<char>((size_t)dm.dr * (dm.dr + dm.d) * es);
  w->xc_f = bp.take<float>((size_t)B * dm.dh); w->x0_f = bp.take<float>((size_t)R * dm.dh);
  w->x1_f = bp.take<float>((size_t)R * dm.dh); w->x2_f = bp.take<float>((size_t)R * dm.dh);
  w->sraw = bp.take<float>((size_t)R * dm.dr); w->hraw = bp.take<float>((size_t)R * dm.dh);
  w->dlogits = bp.take<float>((size_t)R * dm.V);
  w->seg_max = bp.take<float>((size_t)R * 32); w->seg_sum = bp.take<float>((size_t)R * 32);
  w->seg_val = bp.take<float>((size_t)R * 512); w->seg_idx = bp.take<int32_t>((size_t)R * 512);
  w->sel_top = bp.take<unsigned long long>((size_t)R * dm.BW);
  w->lse = bp.take<float>(R); w->cand_val = bp.take<float>((size_t)R * dm.BW);
  w->score_a = bp.take<float>(R); w->score_b = bp.take<float>(R);
  w->cand_idx = bp.take<int32_t>((size_t)R * dm.BW); w->hist_a = bp.take<int32_t>((size_t)R * dm.L);
  w->hist_b = bp.take<int32_t>((size_t)R * dm.L);
  w->tc_partial = bp.take<float>(dm.dtype == RD_DTYPE_BF16 ? tc_partial_floats(TC_MAX_GRID, tc_pick_mt(m_cap)) : 0);
  w->att_scratch = bp.take<float>(dm.dtype == RD_DTYPE_BF16 ? attn_tc_scratch_floats(ATT_MAX_SPLIT_BLOCKS, 1, dm.hd) : 0);
  w->trace = bp.take<unsigned long long>((size_t)TRACE_SLOTS * 8);
  bp.take<char>(256);
}

#define CK(h, expr)                                                                              \
  do {                                                                                           \
    cudaError_t e__ = (expr);                                                                    \
    if (e__ != cudaSuccess) return fail(h, RD_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
    (h)->launches++;                                                                             \
  } while (0)
#define CKRT(h, expr)                                                                            \
  do {                                                                                           \
    cudaError_t e__ = (expr);                                                                    \
    if (e__ != cudaSuccess) return fail(h, RD_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)

// Event pair around one launch when profiling is on (cudaEventCreate happens on first use only).
struct ProfScope {
  rd_handle* h; int cls; cudaStream_t st; bool on;
  ProfScope(rd_handle* h_, int cls_, double bytes, cudaStream_t st_) : h(h_), cls(cls_), st(st_), on(h_->profiling) {
    if (!on) return;
    auto& v = h->ev[cls];
    if (h->ev_used[cls] + 2 > v.size()) {
      cudaEvent_t a, b;
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { on = false; return; }
      v.push_back(a); v.push_back(b);
    }
    cudaEventRecord(v[h->ev_used[cls]], st);
    h->prof_bytes[cls] += bytes;
    h->prof_n[cls]++;
  }
  ~ProfScope() {
    if (!on) return;
    cudaEventRecord(h->ev[cls][h->ev_used[cls] + 1], st);
    h->ev_used[cls] += 2;
  }
};

#define CKP(h, cls, expr)              \
  do {                                 \
    ProfScope ps__(h, cls, 0.0, st);   \
    CK(h, expr);                       \
  } while (0)

// One projection Y = A W^T into the fp32 buffer `raw` (row stride ld_raw); fills `out` for the consumer.
int gemm(rd_handle* h, const void* A, int lda, const void* W, int N, int K, const int32_t* m_total, int m_max, float* raw,
         int ld_raw, GemmOut* out, Chain* chain, cudaStream_t st, int pair = 0) {
  ProfScope ps(h, 0, (double)N * K * esize(h->dm.dtype), st);
  if (h->use_tc) {
    auto iw = h->maps.find(W);
    auto is = h->act_shape.find(A);
    if (iw == h->maps.end() || is == h->act_shape.end() || lda != K || is->second.second != K)
      return fail(h, RD_ERR_STATE, "projection operand without a TMA descriptor");
    const int mt = tc_pick_mt(m_max > 0 ? m_max : 1);
    // activation descriptors: box heights 16..mt in steps of 16 (a launch that has a single row tile picks by the
    // actual row count); made on first use
    const void* amaps[16] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                             nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    // (on CTA pairs each CTA loads half a row tile: heights 8..mt/2 in steps of 8)
    const int pairs = tc_use_pairs(m_max, N, h->tc_grid, h->tc_pairs, h->tc_pairs_min_rows) ? h->tc_pairs : 0;
    const int box_step = pairs ? 8 : 16;
    const int n_maps = mt / 16;
    for (int i = 0; i < n_maps; ++i) {
      const int box_rows = box_step * (i + 1);
      auto key = std::make_pair(A, box_rows);
      auto ia = h->act_maps.find(key);
      if (ia == h->act_maps.end()) {
        TensorMapBox box;
        box.rows = is->second.first; box.cols = K;
        const int rc = tc_make_map(&box, A, (uint64_t)box.rows, (uint64_t)K, (uint32_t)box_rows);
        if (rc) return fail(h, RD_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d for an activation buffer", rc);
        ia = h->act_maps.emplace(key, box).first;
      }
      amaps[i] = &ia->second;
    }
    unsigned long long* tr = nullptr;
    int tr_slot = -1;
    if (h->trace_next >= 0 && h->trace_next < TRACE_SLOTS) {
      if ((int)h->trace_bytes.size() < TRACE_SLOTS) h->trace_bytes.assign(TRACE_SLOTS, 0.0);
      if ((int)h->trace_prefetch.size() < TRACE_SLOTS) h->trace_prefetch.assign(TRACE_SLOTS, 0.0);
      h->trace_bytes[h->trace_next] = (double)N * K * esize(h->dm.dtype);
      tr_slot = h->trace_next;
      tr = h->ws.trace + (size_t)8 * h->trace_next++;
    }
    CK(h, launch_gemm_tc(&iw->second, amaps, N, K, m_total, m_max, raw, ld_raw, h->ws.tc_partial, h->ws.status,
                         h->tc_grid, pairs, h->tc_smem, tr, out, chain, pair, st));
    if (tr_slot >= 0) h->trace_prefetch[tr_slot] = tc_last_prefetch_bytes();
    h->route[pairs ? RD_ROUTE_GEMM_PAIRS : RD_ROUTE_GEMM_ONE_CTA]++;
    return RD_OK;
  }
  if (chain) chain->cut();
  h->route[RD_ROUTE_GEMM_SIMT]++;
  CK(h, launch_gemm_simt(h->dm.dtype, A, lda, W, N, K, m_total, m_max, raw, ld_raw, out, st));
  return RD_OK;
}

// Start of a chained region: counters back in step with the host if an earlier launch was counted but never ran.
int chain_start(rd_handle* h, cudaStream_t st) {
  if (h->chain_dirty) {
    cudaError_t e = h->chain.reset(st);
    if (e != cudaSuccess) return fail(h, RD_ERR_CUDA, "resetting the hand-off counters: %s", cudaGetErrorString(e));
    h->chain_dirty = false;
  }
  h->chain.cut();
  return RD_OK;
}

// ---- context-bound feedback (host side only; never waits)
void fb_invalidate(rd_handle* h) { h->fb_pending[0] = h->fb_pending[1] = false; }

// A copy of the context lengths that has completed bounds every sequence's context by its largest value plus
// whatever the calls enqueued since can have added.
void fb_poll(rd_handle* h) {
  if (!h->fb_host) return;
  for (int s = 0; s < 2; ++s) {
    if (!h->fb_pending[s] || cudaEventQuery(h->fb_event[s]) != cudaSuccess) continue;
    h->fb_pending[s] = false;
    int mx = 0;
    for (int b = 0; b < h->batch; ++b) mx = h->fb_host[(size_t)s * h->dm.B + b] > mx ? h->fb_host[(size_t)s * h->dm.B + b] : mx;
    const long long bound = (long long)mx + (h->fb_growth - h->fb_growth_at[s]);
    if (bound < h->ctx_bound) h->ctx_bound = (int)bound;
  }
  (void)cudaGetLastError();   // cudaEventQuery's cudaErrorNotReady is not an error of this handle
}

// After a call that advanced the contexts by at most `grow` tokens each.
void fb_advance(rd_handle* h, int grow, cudaStream_t st) {
  h->ctx_bound += grow;
  h->fb_growth += grow;
  if (!h->fb_host || (h->fb_calls++ & 7u) != 0u) return;
  const int s = h->fb_next;
  if (h->fb_pending[s]) return;   // that slot's copy is still on its way: try again after the next call
  if (cudaMemcpyAsync(h->fb_host + (size_t)s * h->dm.B, h->ws.ctx, (size_t)h->batch * sizeof(int32_t), cudaMemcpyDeviceToHost, st) !=
          cudaSuccess || cudaEventRecord(h->fb_event[s], st) != cudaSuccess) {
    (void)cudaGetLastError();
    return;
  }
  h->fb_pending[s] = true;
  h->fb_growth_at[s] = h->fb_growth;
  h->fb_next = s ^ 1;
}

char* kv_plane_ptr(rd_handle* h, int layer, int which) {
  return h->kv + ((size_t)(layer * 2 + which)) * h->kv_plane * esize(h->dm.dtype);
}

// Embedding -> n_layers x {attention block, FFN block} -> final norm.  Rows and masks come from the
// row tables in the workspace; results: ws.hidden_f / ws.hidden_t (compact rows).
int forward_layers(rd_handle* h, const uint32_t* mask, int m_max, int n_seq, int rows_per_seq_max, const void* after_w,
                   cudaStream_t st) {
  Workspace& w = h->ws;
  const Dims& dm = h->dm;
  RowTables rt{w.row_tok, w.row_seq, w.row_pos, w.row_slot, w.row_ncache, w.row_local, mask, w.m_total};
  CKP(h, PROF_MISC, launch_embed(dm.dtype, h->w.tok_emb, w.row_tok, w.x, dm.d, dm.V, w.m_total, m_max, w.status, st));
  CKP(h, PROF_MISC, launch_rope_table(w.row_pos, w.rope_tab, dm.hd, dm.theta, w.m_total, m_max, st));
  // attention launch geometry (tensor-core path): tiles of 16 rows per sequence; keys split over CTAs only
  // for long contexts with few tiles
  int row_blocks = 1, n_splits = 1;
  bool att_wide = false, att_shallow = false, att_t5 = false;
  if (h->use_tc) {
    const int rpb = attn_tc_rows_per_block();
    row_blocks = (rows_per_seq_max + rpb - 1) / rpb;
    const int blocks = dm.H * n_seq * row_blocks;
    // The 16-row kernel runs one CTA per SM; past a few waves of them the 64-row kernel (three CTAs per SM, each
    // K/V chunk staged once for four times the rows) takes over.
    static const int wide_waves = getenv("RD_ATT_WIDE") ? atoi(getenv("RD_ATT_WIDE")) : 4;   // tuning toggle
    att_wide = wide_waves < 0 || (wide_waves > 0 && blocks > wide_waves * h->tc_grid);   // negative: always
    static const int t5_ok = getenv("RD_ATT_T5") ? atoi(getenv("RD_ATT_T5")) : 1;   // tuning toggle
    // (its 128-row tiles and 128-key chunks pay off when a sequence brings several hundred rows to the launch -- prompt
    // processing -- or, in a verification pass, when a sequence fills at least half a tile and the context is long
    // enough that a CTA's set-up is spread over eight chunks or more: the batched 7B step takes 17.5 ms this way
    // against 17.9 ms through the 64-row kernel, with 46 of 128 rows used on average.  RD_ATT_T5=2 takes it whenever
    // the 64-row kernel would run.)
    static const int t5_rows = getenv("RD_ATT_T5_ROWS") ? atoi(getenv("RD_ATT_T5_ROWS")) : 64;   // tuning toggle
    const bool t5_pays = rows_per_seq_max >= 512 || (rows_per_seq_max >= t5_rows && h->ctx_bound + rows_per_seq_max >= 1024);
    att_t5 = att_wide && !h->kv_maps.empty() && ((t5_ok == 1 && t5_pays) || t5_ok >= 2);
    if (att_t5) row_blocks = (rows_per_seq_max + attn_t5_rows_per_block() - 1) / attn_t5_rows_per_block();
    else if (att_wide) row_blocks = (rows_per_seq_max + attn_wide_rows_per_block() - 1) / attn_wide_rows_per_block();
    // more 16-row CTAs than SMs (many sequences of a few rows): a two-chunk ring so that three CTAs share an SM
    static const int shallow_ok = getenv("RD_ATT_SHALLOW") ? atoi(getenv("RD_ATT_SHALLOW")) : 1;   // tuning toggle
    att_shallow = shallow_ok && !att_wide && blocks > h->tc_grid;
    n_splits = h->tc_grid / blocks;  // at most one CTA per SM: a second wave would double the time
    // ... and only when a CTA would otherwise walk many chunks: the cross-CTA merge costs several microseconds
    const int max_chunks = (h->ctx_bound + rows_per_seq_max + 63) / 64;
    if (n_splits > (max_chunks + 7) / 8) n_splits = (max_chunks + 7) / 8;
    if (n_splits > 16) n_splits = 16;
    if (n_splits < 1) n_splits = 1;
    while (n_splits > 1 && (long long)blocks * n_splits > ATT_MAX_SPLIT_BLOCKS) --n_splits;
  }
  GemmOut g_qkv, g_o, g_gu, g_dn;
  // inside the layer loop every launch hands over to the next through a counter; the launches before
  // and after it use the grid dependency
  Chain* ch = h->use_tc ? &h->chain : nullptr;
  if (int rc0 = chain_start(h, st)) return rc0;
  for (int l = 0; l < dm.n_layers; ++l) {
    // attention block: (x += down of the previous layer) -> norm -> QKV -> rotary + KV write -> attention -> O
    CKP(h, PROF_NORM, launch_rmsnorm(dm.dtype, w.x, l ? &g_dn : nullptr, h->attn_norm[l], w.a_t, nullptr, dm.d, dm.eps,
                                     w.m_total, m_max, ch, st));
    int rc = gemm(h, w.a_t, dm.d, h->wqkv[l], 3 * dm.d, dm.d, w.m_total, m_max, w.qkv, 3 * dm.d, &g_qkv, ch, st, /*pair=*/1);
    if (rc) return rc;
    CKP(h, PROF_ROPE, launch_rope_kv(dm.dtype, w.qkv, g_qkv, kv_plane_ptr(h, l, 0), kv_plane_ptr(h, l, 1), w.rope_tab, rt, dm,
                                     m_max, w.status, ch, st));
    {
      ProfScope ps(h, 1, 0.0, st);
      h->route[!h->use_tc ? RD_ROUTE_ATT_FP32 : att_t5 ? RD_ROUTE_ATT_ROWS128_TC5 : att_wide ? RD_ROUTE_ATT_ROWS64
               : att_shallow ? RD_ROUTE_ATT_ROWS16_SHALLOW : RD_ROUTE_ATT_ROWS16]++;
      if (h->use_tc && !att_t5 && !att_wide && n_splits > 1) h->route[RD_ROUTE_ATT_KEY_SPLIT]++;
      if (h->use_tc && att_t5)
        CK(h, launch_attention_t5(h->kv_maps[(size_t)l * 2].bytes, h->kv_maps[(size_t)l * 2 + 1].bytes, w.qkv, w.attn_t, rt, w.seq_off, h->att_seq_order, dm, n_seq,
                                  row_blocks, w.status, ch, st));
      else if (h->use_tc && att_wide)
        CK(h, launch_attention_wide(w.qkv, kv_plane_ptr(h, l, 0), kv_plane_ptr(h, l, 1), w.attn_t, rt, w.seq_off, dm, n_seq,
                                    row_blocks, ch, st));
      else if (h->use_tc)
        CK(h, launch_attention_tc(w.qkv, kv_plane_ptr(h, l, 0), kv_plane_ptr(h, l, 1), w.attn_t, rt, w.seq_off, dm, n_seq,
                                  row_blocks, n_splits, w.att_scratch, w.att_counters,
                                  (h->trace_next >= 0 && h->trace_next < TRACE_SLOTS) ? w.trace + (size_t)8 * h->trace_next++ : nullptr, ch,
                                  att_shallow ? 1 : 0, st));
      else
        CK(h, launch_attention(dm.dtype, w.qkv, kv_plane_ptr(h, l, 0), kv_plane_ptr(h, l, 1), w.attn_t, rt, dm, m_max, st));
    }
    rc = gemm(h, w.attn_t, dm.d, h->wo[l], dm.d, dm.d, w.m_total, m_max, w.proj_d, dm.d, &g_o, ch, st, /*pair=*/1);
    if (rc) return rc;
    // FFN block: (x += O) -> norm -> gate|up -> SwiGLU -> down
    CKP(h, PROF_NORM, launch_rmsnorm(dm.dtype, w.x, &g_o, h->ffn_norm[l], w.a_t, nullptr, dm.d, dm.eps, w.m_total, m_max, ch, st));
    rc = gemm(h, w.a_t, dm.d, h->w_gate_up[l], 2 * dm.F, dm.d, w.m_total, m_max, w.gu, 2 * dm.F, &g_gu, ch, st, /*pair=*/1);
    if (rc) return rc;
    CKP(h, PROF_SWIGLU, launch_swiglu(dm.dtype, g_gu, w.act_t, dm.F, w.m_total, m_max, w.status, ch, st));
    rc = gemm(h, w.act_t, dm.F, h->w_down[l], dm.d, dm.F, w.m_total, m_max, w.proj_d, dm.d, &g_dn, ch, st, /*pair=*/1);
    if (rc) return rc;
  }
  CKP(h, PROF_NORM, launch_rmsnorm(dm.dtype, w.x, &g_dn, h->w.final_norm, w.hidden_t, w.hidden_f, dm.d, dm.eps, w.m_total,
                                   m_max, ch, st));
  h->chain.cut();
  return RD_OK;
}

int check_stepable(rd_handle* h) {
  if (!h) return RD_ERR_INVALID_ARG;
  if (!h->prefilled) return fail(h, RD_ERR_STATE, "no state: call redrafter_prefill or redrafter_set_state first");
  fb_poll(h);
  if (h->ctx_bound + h->dm.NMAX > h->dm.max_ctx)
    return fail(h, RD_ERR_CAPACITY, "context bound %d + %d packed rows exceeds max_ctx %d", h->ctx_bound, h->dm.NMAX,
                h->dm.max_ctx);
  return RD_OK;
}

int do_draft(rd_handle* h, cudaStream_t st, int32_t* beams, float* scores) {
  Workspace& w = h->ws;
  const Dims& dm = h->dm;
  const int B = h->batch, R = B * dm.BW;
  CKP(h, PROF_DRAFT_SMALL, launch_draft_init(dm.dtype, h->w.tok_emb, w.root, w.h, w.xc_t, w.xc_f, w.se_t, dm, B, w.status, st));
  if (dm.L > 1) CKP(h, PROF_DRAFT_SMALL, launch_fill_h(dm.dtype, w.h, w.x0_t, w.x0_f, dm, B, st));
  float *sc_in = w.score_a, *sc_out = w.score_b;
  int32_t *hi_in = w.hist_a, *hi_out = w.hist_b;
  GemmOut g;
  // the calls' launches hand over to each other through counters (tensor-core path)
  Chain* ch = h->use_tc ? &h->chain : nullptr;
  if (int rc0 = chain_start(h, st)) return rc0;
  for (int call = 1; call <= dm.L; ++call) {
    const int rows = call == 1 ? B : R;
    const int32_t* mt = call == 1 ? w.one_b : w.one_r;
    const void* xin_t = call == 1 ? w.xc_t : w.x0_t;
    const float* xin_f = call == 1 ? w.xc_f : w.x0_f;
    if (call > 1) {
      // s_t = SiLU([U W][s_{t-1}; e_t] + b), written into the first d_rnn columns of x0 = [s_t, h]
      int rc = gemm(h, w.se_t, dm.dr + dm.d, w.uw, dm.dr, dm.dr + dm.d, mt, rows, w.sraw, dm.dr, &g, ch, st, /*pair=*/1);
      if (rc) return rc;
      CKP(h, PROF_DRAFT_SMALL, launch_act(dm.dtype, g, h->w.rnn_b, nullptr, 0, w.x0_f, w.x0_t, dm.dh, dm.dr, mt, rows, ch, st));
    }
    for (int l = 0; l < dm.n_head_layers; ++l) {
      float* of = (l & 1) ? w.x2_f : w.x1_f;
      void* ot = (l & 1) ? w.x2_t : w.x1_t;
      int rc = gemm(h, xin_t, dm.dh, h->head_w[l], dm.dh, dm.dh, mt, rows, w.hraw, dm.dh, &g, ch, st, /*pair=*/1);
      if (rc) return rc;
      CKP(h, PROF_DRAFT_SMALL, launch_act(dm.dtype, g, h->head_b[l], xin_f, dm.dh, of, ot, dm.dh, dm.dh, mt, rows, ch, st));
      xin_t = ot; xin_f = of;
    }
    int rc = gemm(h, xin_t, dm.dh, h->w.draft_out, dm.V, dm.dh, mt, rows, w.dlogits, dm.V, &g, ch, st, /*pair=*/1);
    if (rc) return rc;
    CKP(h, PROF_DRAFT_SMALL, launch_draft_select(dm.dtype, g, call, w.lse, w.cand_val, w.cand_idx, sc_in, sc_out, hi_in, hi_out,
                                                 h->w.tok_emb, w.x0_f, dm.dh, w.se_t, dm, B, beams, scores, w.sel_counters, mt,
                                                 (h->trace_next >= 0 && h->trace_next < TRACE_SLOTS) ? w.trace + (size_t)8 * h->trace_next++ : nullptr,
                                                 SelectScratch{h->use_tc ? w.seg_max : nullptr, w.seg_sum, w.seg_val, w.seg_idx, h->tc_grid, w.sel_top}, ch, st));
    if (h->use_tc && draft_select_segments(dm, rows, h->tc_grid) > 0) h->launches += 2;   // that selection is three launches
    float* tf = sc_in; sc_in = sc_out; sc_out = tf;
    int32_t* ti = hi_in; hi_in = hi_out; hi_out = ti;
  }
  h->chain.cut();
  return RD_OK;
}

int do_verify(rd_handle* h, const rd_packed& pk, cudaStream_t st, int32_t* argmax, float* hidden, float* logits) {
  Workspace& w = h->ws;
  const Dims& dm = h->dm;
  const int B = h->batch, m_max = B * dm.NMAX;
  CKP(h, PROF_MISC, launch_build_rows_tree(pk, w.ctx, w.row_tok, w.row_seq, w.row_pos, w.row_slot, w.row_ncache, w.row_local,
                               w.row_out_index, w.seq_off, w.seq_order, w.m_total, dm, B, w.status, st));
  h->att_seq_order = B <= 1024 ? w.seq_order : nullptr;   // the row tables of this pass carry the sequences' order
  int rc = forward_layers(h, pk.mask, m_max, B, dm.NMAX, h->w.lm_head, st);
  h->att_seq_order = nullptr;
  if (rc) return rc;
  GemmOut g;
  rc = gemm(h, w.hidden_t, dm.d, h->w.lm_head, dm.V, dm.d, w.m_total, m_max, w.logits, dm.V, &g, nullptr, st, /*pair=*/1);
  if (rc) return rc;
  CKP(h, PROF_MISC, launch_fill_i32(argmax, -1, B * dm.NMAX, st));
  CKP(h, PROF_MISC, launch_argmax_rows(w.logits, g, dm.V, argmax, w.row_out_index, w.m_total, m_max, h->sampling, w.row_seq, w.row_pos, 1, st));
  if (hidden) CKP(h, PROF_MISC, launch_scatter_rows(w.hidden_f, dm.d, hidden, w.row_out_index, w.m_total, m_max, st));
  if (logits) CK(h, launch_scatter_rows(w.logits, dm.V, logits, w.row_out_index, w.m_total, m_max, st));
  return RD_OK;
}

}  // namespace

// One warp whose first thread waits, bounded, on a hand-off counter value that no launch will ever produce.
__global__ void selftest_wait_kernel(rd::ChainSync cs) {
  if (threadIdx.x == 0) rd::chain_wait_thread(cs);
}

extern "C" {

size_t redrafter_workspace_bytes(const rd_config* cfg) {
  Dims dm;
  if (!make_dims(cfg, &dm) || !shape_ok(dm)) return 0;
  Bump bp{nullptr, 0};
  Workspace w;
  carve(bp, dm, m_cap_of(dm), &w);
  return bp.off;
}

size_t redrafter_kv_bytes(const rd_config* cfg) {
  Dims dm;
  if (!make_dims(cfg, &dm)) return 0;
  return (size_t)dm.n_layers * 2 * dm.B * dm.H * (size_t)dm.max_ctx * dm.hd * esize(dm.dtype);
}

int redrafter_init(const rd_config* cfg, const rd_weights* wt, void* kv_cache, size_t kv_bytes, void* workspace,
                   size_t ws_bytes, rd_handle** out) {
  if (!cfg || !wt || !kv_cache || !workspace || !out) return RD_ERR_INVALID_ARG;
  *out = nullptr;
  Dims dm;
  if (!make_dims(cfg, &dm)) return RD_ERR_INVALID_ARG;
  if (!shape_ok(dm)) return RD_ERR_SHAPE;
  if (((uintptr_t)kv_cache | (uintptr_t)workspace) & 255) return RD_ERR_INVALID_ARG;
  if (kv_bytes < redrafter_kv_bytes(cfg) || ws_bytes < redrafter_workspace_bytes(cfg)) return RD_ERR_CAPACITY;
  if (!wt->tok_emb || !wt->final_norm || !wt->lm_head || !wt->attn_norm || !wt->wqkv || !wt->wo || !wt->ffn_norm ||
      !wt->w_gate_up || !wt->w_down || !wt->rnn_u || !wt->rnn_w || !wt->rnn_b || !wt->draft_out ||
      (dm.n_head_layers && (!wt->head_w || !wt->head_b)))
    return RD_ERR_INVALID_ARG;
  rd_handle* h = new (std::nothrow) rd_handle();
  if (!h) return RD_ERR_INVALID_ARG;
  h->cfg = *cfg; h->dm = dm; h->m_cap = m_cap_of(dm);
  h->kv = (char*)kv_cache;
  h->kv_plane = (size_t)dm.B * dm.H * (size_t)dm.max_ctx * dm.hd;
  h->w = *wt;
  for (int l = 0; l < dm.n_layers; ++l) {
    h->attn_norm.push_back(wt->attn_norm[l]); h->wqkv.push_back(wt->wqkv[l]); h->wo.push_back(wt->wo[l]);
    h->ffn_norm.push_back(wt->ffn_norm[l]); h->w_gate_up.push_back(wt->w_gate_up[l]); h->w_down.push_back(wt->w_down[l]);
    if (!wt->attn_norm[l] || !wt->wqkv[l] || !wt->wo[l] || !wt->ffn_norm[l] || !wt->w_gate_up[l] || !wt->w_down[l]) {
      delete h;
      return RD_ERR_INVALID_ARG;
    }
  }
  for (int l = 0; l < dm.n_head_layers; ++l) {
    h->head_w.push_back(wt->head_w[l]); h->head_b.push_back(wt->head_b[l]);
    if (!wt->head_w[l] || !wt->head_b[l]) { delete h; return RD_ERR_INVALID_ARG; }
  }
  Bump bp{(char*)workspace, 0};
  carve(bp, dm, h->m_cap, &h->ws);
  h->use_tc = dm.dtype == RD_DTYPE_BF16 && !(cfg->flags & RD_FLAG_FORCE_SIMT);
  {
    cudaError_t ce = elementwise_prepare(dm.dtype);
    if (ce == cudaSuccess) ce = drafter_prepare(dm.dtype);
    if (ce != cudaSuccess) return init_fail(h, RD_ERR_CUDA, "kernel set-up: %s", cudaGetErrorString(ce));
  }
  h->tc_pairs = 0; h->tc_pairs_avail = 0; h->tc_pairs_min_rows = 1024; h->tc_pairs_prefill = false;
  if (h->use_tc) {
    int dev = 0, sms = 0;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce == cudaSuccess) ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (ce == cudaSuccess) ce = tc_prepare(&h->tc_smem, &h->tc_pairs_avail);
    if (ce == cudaSuccess) ce = attn_tc_prepare(dm.hd, dm.MW);
    if (ce == cudaSuccess) ce = attn_wide_prepare(dm.hd, dm.MW);
    if (ce == cudaSuccess) ce = attn_t5_prepare(dm.hd, dm.MW);
    if (ce != cudaSuccess || sms <= 0)
      return init_fail(h, RD_ERR_CUDA, "tensor-core path set-up: %s", cudaGetErrorString(ce));
    h->tc_grid = sms < TC_MAX_GRID ? sms : TC_MAX_GRID;
    // CTA-pair projections (tuning toggles, read when the handle is made): from a bound of 1024 rows in decode steps
    // (measured: 1-4 % of the step from about 650 packed rows; with bounds around 650 rows, 300-420 rows present, the
    // one-CTA kernel, which starts earlier and has shorter tails, is 3-5 % ahead); RD_TC_CTA2=0 never, RD_TC_CTA2_MIN the row bound, RD_TC_CTA2_PREFILL=1 also in prompt passes.
    if (getenv("RD_TC_CTA2") && atoi(getenv("RD_TC_CTA2")) == 0) h->tc_pairs_avail = 0;
    h->tc_pairs_min_rows = getenv("RD_TC_CTA2_MIN") ? atoi(getenv("RD_TC_CTA2_MIN")) : 1024;
    h->tc_pairs_prefill = getenv("RD_TC_CTA2_PREFILL") && atoi(getenv("RD_TC_CTA2_PREFILL")) != 0;
    h->tc_pairs = h->tc_pairs_avail;
    if (attn_t5_supported(dm.hd)) {
      // The tensor-core attention multiplies masked-out V rows by exact zeros: the cache has to hold finite values.
      ce = cudaMemset(h->kv, 0, (size_t)dm.n_layers * 2 * h->kv_plane * esize(dm.dtype));
      if (ce != cudaSuccess) return init_fail(h, RD_ERR_CUDA, "clearing the KV cache: %s", cudaGetErrorString(ce));
      h->kv_maps.resize((size_t)dm.n_layers * 2);
      for (int l = 0; l < dm.n_layers; ++l)
        for (int which = 0; which < 2; ++which)
          if (tc_make_map(h->kv_maps[(size_t)l * 2 + which].bytes, kv_plane_ptr(h, l, which), (uint64_t)dm.B * dm.H * dm.max_ctx, dm.hd, 128) != 0)
            return init_fail(h, RD_ERR_CUDA, "tensor map of the KV cache (layer %d)", l);
    }
    if (dm.d % 8 || dm.F % 8 || dm.dh % 8) return init_fail(h, RD_ERR_SHAPE, "bf16 needs d_model, d_ffn multiples of 8");
    bool ok = true;
    int failed_rc = 0;
    const void* failed_ptr = nullptr;
    auto add_w = [&](const void* p, int N, int K) {
      if (!ok) return;
      TensorMapBox& box = h->maps[p];
      box.rows = N; box.cols = K;
      failed_rc = tc_make_map(&box, p, (uint64_t)N, (uint64_t)K, (uint32_t)tc_weight_box_rows());
      if (failed_rc) { ok = false; failed_ptr = p; }
    };
    auto add_a = [&](const void* p, int rows, int K) { h->act_shape[p] = std::make_pair(rows, K); };
    for (int l = 0; l < dm.n_layers; ++l) {
      add_w(h->wqkv[l], 3 * dm.d, dm.d); add_w(h->wo[l], dm.d, dm.d);
      add_w(h->w_gate_up[l], 2 * dm.F, dm.d); add_w(h->w_down[l], dm.d, dm.F);
    }
    add_w(wt->lm_head, dm.V, dm.d); add_w(h->ws.uw, dm.dr, dm.dr + dm.d);
    for (int l = 0; l < dm.n_head_layers; ++l) add_w(h->head_w[l], dm.dh, dm.dh);
    add_w(wt->draft_out, dm.V, dm.dh);
    const Workspace& w = h->ws;
    const int R = dm.B * dm.BW;
    add_a(w.a_t, h->m_cap, dm.d); add_a(w.attn_t, h->m_cap, dm.d); add_a(w.act_t, h->m_cap, dm.F);
    add_a(w.hidden_t, h->m_cap, dm.d); add_a(w.h_t, dm.B, dm.d);
    add_a(w.xc_t, dm.B, dm.dh); add_a(w.x0_t, R, dm.dh); add_a(w.x1_t, R, dm.dh); add_a(w.x2_t, R, dm.dh);
    add_a(w.se_t, R, dm.dr + dm.d);
    if (!ok) return init_fail(h, RD_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d for operand %p", failed_rc, failed_ptr);
  }
  h->prefilled = false; h->batch = dm.B; h->ctx_bound = 0; h->launches = 0; h->err[0] = 0;
  for (int i = 0; i < RD_ROUTE_COUNT; ++i) h->route[i] = 0;
  h->sampling = Sampling{0.0f, 0u, 0u};
  h->profiling = false;
  h->trace_next = -1;
  h->chain.ctr = h->ws.chain_ctr; h->chain.status = h->ws.status;
  h->chain.trace_base = h->ws.trace; h->chain.trace_next = &h->trace_next; h->chain.trace_cap = TRACE_SLOTS;
  h->chain.enabled = !(getenv("RD_CHAIN") && atoi(getenv("RD_CHAIN")) == 0);
  h->chain_dirty = false;
  h->device = 0;
  (void)cudaGetDevice(&h->device);
  // pinned host memory and two events for the context-bound feedback (host resources; no device memory)
  h->fb_host = nullptr; h->fb_pending[0] = h->fb_pending[1] = false; h->fb_growth = 0; h->fb_next = 0; h->fb_calls = 0;
  h->fb_event[0] = h->fb_event[1] = nullptr;
  if (cudaHostAlloc((void**)&h->fb_host, (size_t)2 * dm.B * sizeof(int32_t), cudaHostAllocDefault) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->fb_event[0], cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->fb_event[1], cudaEventDisableTiming) != cudaSuccess) {
    (void)cudaGetLastError();
    if (h->fb_host) cudaFreeHost(h->fb_host);
    h->fb_host = nullptr;   // the bound then simply grows by 1 + L per step until the caller refreshes it
  }
  for (int c = 0; c < PROF_CLASSES; ++c) { h->ev_used[c] = 0; h->prof_ms[c] = 0; h->prof_bytes[c] = 0; h->prof_n[c] = 0; }
  // clear the state and the constants the kernels read from device memory
  cudaError_t e = cudaMemsetAsync(workspace, 0, (size_t)((char*)h->ws.x - (char*)workspace), 0);
  // [U W]: the RNN's two matrices side by side, so that s_t needs one projection over [s ; e]
  const size_t es_ = esize(dm.dtype);
  if (e == cudaSuccess)
    e = cudaMemcpy2DAsync(h->ws.uw, (size_t)(dm.dr + dm.d) * es_, wt->rnn_u, (size_t)dm.dr * es_, (size_t)dm.dr * es_, dm.dr,
                          cudaMemcpyDeviceToDevice, 0);
  if (e == cudaSuccess)
    e = cudaMemcpy2DAsync((char*)h->ws.uw + (size_t)dm.dr * es_, (size_t)(dm.dr + dm.d) * es_, wt->rnn_w, (size_t)dm.d * es_,
                          (size_t)dm.d * es_, dm.dr, cudaMemcpyDeviceToDevice, 0);
  if (e == cudaSuccess) e = cudaStreamSynchronize(0);
  if (e != cudaSuccess) { delete h; return RD_ERR_CUDA; }
  *out = h;
  return RD_OK;
}

int redrafter_destroy(rd_handle* h) {
  if (!h) return RD_ERR_INVALID_ARG;
  for (int c = 0; c < PROF_CLASSES; ++c)
    for (cudaEvent_t e : h->ev[c]) cudaEventDestroy(e);
  if (h->fb_host) {
    for (int s = 0; s < 2; ++s)
      if (h->fb_pending[s]) cudaEventSynchronize(h->fb_event[s]);   // a copy into the pinned buffer may still be in flight
    cudaFreeHost(h->fb_host);
  }
  for (int s = 0; s < 2; ++s)
    if (h->fb_event[s]) cudaEventDestroy(h->fb_event[s]);
  delete h;
  return RD_OK;
}

const char* redrafter_last_error(const rd_handle* h) { return h ? h->err : g_init_err; }

int64_t redrafter_launch_count(const rd_handle* h) { return h ? h->launches : 0; }

int redrafter_last_logits(rd_handle* h, void* stream, float* out, int32_t rows) {
  if (!h || !out || rows <= 0 || rows > h->dm.B * h->dm.NMAX) return RD_ERR_INVALID_ARG;
  CKRT(h, cudaMemcpyAsync(out, h->ws.logits, (size_t)rows * h->dm.V * sizeof(float), cudaMemcpyDeviceToDevice,
                          (cudaStream_t)stream));
  return RD_OK;
}

int redrafter_route_counts(const rd_handle* h, int64_t* out, int32_t n) {
  if (!h || !out || n < 0 || n > RD_ROUTE_COUNT) return RD_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) out[i] = h->route[i];
  return RD_OK;
}

static int set_row_counts(rd_handle* h, cudaStream_t st) {
  CK(h, launch_fill_i32(h->ws.one_b, h->batch, 1, st));
  CK(h, launch_fill_i32(h->ws.one_r, h->batch * h->dm.BW, 1, st));
  return RD_OK;
}

int redrafter_prefill(rd_handle* h, const int32_t* tokens, const int32_t* prompt_len, int32_t max_prompt, int32_t batch,
                      void* stream) {
  if (!h || !tokens || !prompt_len) return RD_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const Dims& dm = h->dm;
  Workspace& w = h->ws;
  if (batch <= 0 || batch > dm.B) return fail(h, RD_ERR_INVALID_ARG, "batch %d outside [1, %d]", batch, dm.B);
  int longest = 0;
  for (int b = 0; b < batch; ++b) {
    if (prompt_len[b] <= 0 || prompt_len[b] > max_prompt) return fail(h, RD_ERR_INVALID_ARG, "prompt_len[%d] = %d", b, prompt_len[b]);
    if (prompt_len[b] + dm.NMAX > dm.max_ctx) return fail(h, RD_ERR_CAPACITY, "prompt %d of length %d leaves no room for a step", b, prompt_len[b]);
    longest = prompt_len[b] > longest ? prompt_len[b] : longest;
  }
  h->batch = batch;
  int rc = set_row_counts(h, st);
  if (rc) return rc;
  // passes of up to m_cap rows; a sequence's rows may span passes (its earlier rows are in the cache by then)
  const int cap = h->m_cap;
  std::vector<int32_t> tok(cap), seq(cap), pos(cap), ncache(cap), local(cap), last(batch), soff(batch + 1), count(batch);
  int b = 0, done = 0;  // next sequence, tokens of it already processed
  while (b < batch) {
    int m = 0, longest_run = 0;
    for (int i = 0; i < batch; ++i) { last[i] = -1; count[i] = 0; }
    while (b < batch && m < cap) {
      const int take = (prompt_len[b] - done) < (cap - m) ? (prompt_len[b] - done) : (cap - m);
      for (int i = 0; i < take; ++i) {
        tok[m] = tokens[(size_t)b * max_prompt + done + i];
        seq[m] = b; pos[m] = done + i; ncache[m] = done + i + 1; local[m] = 0;
        ++m;
      }
      count[b] = take;
      if (take > longest_run) longest_run = take;
      done += take;
      if (done == prompt_len[b]) { last[b] = m - 1; ++b; done = 0; }
    }
    // the sequences of a pass are consecutive and their rows contiguous from row 0
    soff[0] = 0;
    for (int i = 0; i < batch; ++i) soff[i + 1] = soff[i] + count[i];
    const size_t nb = (size_t)m * sizeof(int32_t);
    CKRT(h, cudaMemcpyAsync(w.row_tok, tok.data(), nb, cudaMemcpyHostToDevice, st));
    CKRT(h, cudaMemcpyAsync(w.row_seq, seq.data(), nb, cudaMemcpyHostToDevice, st));
    CKRT(h, cudaMemcpyAsync(w.row_pos, pos.data(), nb, cudaMemcpyHostToDevice, st));
    CKRT(h, cudaMemcpyAsync(w.row_slot, pos.data(), nb, cudaMemcpyHostToDevice, st));
    CKRT(h, cudaMemcpyAsync(w.row_ncache, ncache.data(), nb, cudaMemcpyHostToDevice, st));
    CKRT(h, cudaMemcpyAsync(w.row_local, local.data(), nb, cudaMemcpyHostToDevice, st));
    CKRT(h, cudaMemcpyAsync(w.last_row, last.data(), batch * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    CKRT(h, cudaMemcpyAsync(w.seq_off, soff.data(), (batch + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    CKRT(h, cudaMemcpyAsync(w.m_total, &m, sizeof(int32_t), cudaMemcpyHostToDevice, st));
    CKRT(h, cudaStreamSynchronize(st));  // the host staging vectors are reused by the next pass
    h->ctx_bound = longest;  // bound of the key extent for this pass
    // Prompt passes keep the one-CTA projection: their rows fill 256-row tiles exactly, projection plus consumer
    // take the same time with either kernel (the fp32 intermediate bounds the pair), and the CTA pairs start later.
    if (!h->tc_pairs_prefill) h->tc_pairs = 0;
    rc = forward_layers(h, nullptr, m, batch, longest_run, nullptr, st);
    h->tc_pairs = h->tc_pairs_avail;
    if (rc) return rc;
    CK(h, launch_prefill_finish(w.hidden_f, w.last_row, w.h, dm.d, batch, st));
  }
  // root token: the greedy token after the prompt = argmax(lm_head h)
  CK(h, launch_cast_rows(dm.dtype, w.h, w.h_t, batch * dm.d, st));
  GemmOut g;
  rc = gemm(h, w.h_t, dm.d, h->w.lm_head, dm.V, dm.d, w.one_b, batch, w.logits, dm.V, &g, nullptr, st);
  if (rc) return rc;
  CKRT(h, cudaMemcpyAsync(w.ctx, prompt_len, batch * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  // row b is sequence b's last prompt row: the root is the token at position prompt_len[b]
  CK(h, launch_argmax_rows(w.logits, g, dm.V, w.root, nullptr, w.one_b, batch, h->sampling, nullptr, w.ctx, 0, st));
  h->prefilled = true;
  h->ctx_bound = longest;
  fb_invalidate(h);
  return RD_OK;
}

int redrafter_draft(rd_handle* h, void* stream, int32_t* beams, float* scores) {
  int rc = check_stepable(h);
  if (rc) return rc;
  if (!beams) return fail(h, RD_ERR_INVALID_ARG, "beams is null");
  return do_draft(h, (cudaStream_t)stream, beams, scores);
}

static bool packed_ok(const rd_packed* p) {
  return p && p->tokens && p->n && p->unpack && p->pos && p->mask && p->parent;
}

int redrafter_pack(rd_handle* h, const int32_t* beams, void* stream, const rd_packed* out) {
  int rc = check_stepable(h);
  if (rc) return rc;
  if (!beams || !packed_ok(out)) return fail(h, RD_ERR_INVALID_ARG, "null beams or packed member");
  cudaStream_t st = (cudaStream_t)stream;
  CK(h, launch_pack(beams, h->ws.root, h->ws.ctx, *out, h->dm, h->batch, (h->cfg.flags & RD_FLAG_NO_TREE) ? 1 : 0, st));
  return RD_OK;
}

int redrafter_verify(rd_handle* h, const rd_packed* packed, void* stream, int32_t* argmax, float* hidden, float* logits) {
  int rc = check_stepable(h);
  if (rc) return rc;
  if (!packed_ok(packed) || !argmax) return fail(h, RD_ERR_INVALID_ARG, "null packed member or argmax");
  return do_verify(h, *packed, (cudaStream_t)stream, argmax, hidden, logits);
}

int redrafter_accept(rd_handle* h, const int32_t* beams, const rd_packed* packed, const int32_t* argmax,
                     const float* hidden, void* stream, const rd_accept_out* out) {
  int rc = check_stepable(h);
  if (rc) return rc;
  if (!beams || !packed_ok(packed) || !argmax || !hidden) return fail(h, RD_ERR_INVALID_ARG, "null argument");
  Workspace& w = h->ws;
  rd_accept_out o{};
  if (out) o = *out;
  CK(h, launch_accept(h->dm.dtype, beams, *packed, argmax, hidden, h->kv, w.ctx, w.root, w.h, o, w.n_accept, w.best,
                      w.ctx_prev, h->dm, h->batch, w.status, (cudaStream_t)stream));
  h->launches++;  // accept + compaction
  fb_advance(h, 1 + h->dm.L, (cudaStream_t)stream);
  return RD_OK;
}

int redrafter_accept_static(rd_handle* h, const int32_t* beams, const rd_packed* packed, const int32_t* argmax,
                            const float* hidden, void* stream, const rd_accept_out* out) {
  int rc = check_stepable(h);
  if (rc) return rc;
  if (!beams || !packed_ok(packed) || !argmax || !hidden) return fail(h, RD_ERR_INVALID_ARG, "null argument");
  int dev_now = -1;
  if (cudaGetDevice(&dev_now) != cudaSuccess || dev_now != h->device)
    return fail(h, RD_ERR_STATE, "current device %d is not the device %d this handle was made on", dev_now, h->device);
  if (h->batch > accept_static_max_batch())
    return fail(h, RD_ERR_CAPACITY, "batch %d exceeds the %d sequences the built-in scratch holds", h->batch,
                accept_static_max_batch());
  int32_t *n_accept = nullptr, *best = nullptr, *ctx_prev = nullptr;
  cudaError_t e = accept_static_scratch(&n_accept, &best, &ctx_prev);
  if (e != cudaSuccess) return fail(h, RD_ERR_CUDA, "built-in scratch: %s", cudaGetErrorString(e));
  Workspace& w = h->ws;
  rd_accept_out o{};
  if (out) o = *out;
  CK(h, launch_accept(h->dm.dtype, beams, *packed, argmax, hidden, h->kv, w.ctx, w.root, w.h, o, n_accept, best, ctx_prev,
                      h->dm, h->batch, w.status, (cudaStream_t)stream));
  h->launches++;  // accept + compaction
  fb_advance(h, 1 + h->dm.L, (cudaStream_t)stream);
  return RD_OK;
}

int redrafter_step(rd_handle* h, const int32_t* planted_beams, void* stream, const rd_accept_out* out) {
  int rc = check_stepable(h);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  Workspace& w = h->ws;
  rc = do_draft(h, st, w.beams, w.scores);
  if (rc) return rc;
  const int32_t* beams = planted_beams ? planted_beams : w.beams;
  CKP(h, PROF_PACK_ACCEPT, launch_pack(beams, w.root, w.ctx, w.pk, h->dm, h->batch, (h->cfg.flags & RD_FLAG_NO_TREE) ? 1 : 0, st));
  rc = do_verify(h, w.pk, st, w.argmax_p, w.hidden_p, nullptr);
  if (rc) return rc;
  rd_accept_out o{};
  if (out) o = *out;
  CKP(h, PROF_PACK_ACCEPT, launch_accept(h->dm.dtype, beams, w.pk, w.argmax_p, w.hidden_p, h->kv, w.ctx, w.root, w.h, o, w.n_accept,
                      w.best, w.ctx_prev, h->dm, h->batch, w.status, st));
  h->launches++;
  fb_advance(h, 1 + h->dm.L, st);
  return RD_OK;
}

int redrafter_ar_step(rd_handle* h, void* stream, int32_t* token) {
  if (!h) return RD_ERR_INVALID_ARG;
  if (!h->prefilled) return fail(h, RD_ERR_STATE, "no state: call redrafter_prefill or redrafter_set_state first");
  fb_poll(h);
  if (h->ctx_bound + 1 > h->dm.max_ctx) return fail(h, RD_ERR_CAPACITY, "KV cache full");
  cudaStream_t st = (cudaStream_t)stream;
  Workspace& w = h->ws;
  const Dims& dm = h->dm;
  const int B = h->batch;
  CK(h, launch_build_rows_ar(w.root, w.ctx, w.row_tok, w.row_seq, w.row_pos, w.row_slot, w.row_ncache, w.row_local,
                             w.row_out_index, w.seq_off, w.m_total, dm, B, w.status, st));
  int rc = forward_layers(h, nullptr, B, B, 1, h->w.lm_head, st);
  if (rc) return rc;
  GemmOut g;
  rc = gemm(h, w.hidden_t, dm.d, h->w.lm_head, dm.V, dm.d, w.m_total, B, w.logits, dm.V, &g, nullptr, st);
  if (rc) return rc;
  CK(h, launch_argmax_rows(w.logits, g, dm.V, w.argmax_c, nullptr, w.m_total, B, h->sampling, w.row_seq, w.row_pos, 1, st));
  CK(h, launch_ar_finish(w.argmax_c, w.hidden_f, w.ctx, w.root, w.h, token, dm, B, st));
  fb_advance(h, 1, st);
  return RD_OK;
}

int redrafter_set_sampling(rd_handle* h, float temperature, uint64_t seed) {
  if (!h) return RD_ERR_INVALID_ARG;
  if (!(temperature >= 0.0f) || !std::isfinite(temperature)) return fail(h, RD_ERR_INVALID_ARG, "temperature %g", (double)temperature);
  h->sampling.inv_t = temperature > 0.0f ? 1.0f / temperature : 0.0f;
  h->sampling.k0 = (uint32_t)(seed & 0xffffffffull);
  h->sampling.k1 = (uint32_t)(seed >> 32);
  return RD_OK;
}

int redrafter_get_state(rd_handle* h, void* stream, int32_t* ctx, int32_t* root, float* hvec) {
  if (!h) return RD_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t B = h->batch;
  if (ctx) CKRT(h, cudaMemcpyAsync(ctx, h->ws.ctx, B * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  if (root) CKRT(h, cudaMemcpyAsync(root, h->ws.root, B * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  if (hvec) CKRT(h, cudaMemcpyAsync(hvec, h->ws.h, B * h->dm.d * sizeof(float), cudaMemcpyDeviceToDevice, st));
  return RD_OK;
}

int redrafter_set_state(rd_handle* h, void* stream, const int32_t* ctx, const int32_t* root, const float* hvec,
                        int32_t batch) {
  if (!h) return RD_ERR_INVALID_ARG;
  if (batch <= 0 || batch > h->dm.B) return fail(h, RD_ERR_INVALID_ARG, "batch %d outside [1, %d]", batch, h->dm.B);
  cudaStream_t st = (cudaStream_t)stream;
  h->batch = batch;
  int rc = set_row_counts(h, st);
  if (rc) return rc;
  const size_t B = batch;
  if (ctx) {
    CKRT(h, cudaMemcpyAsync(h->ws.ctx, ctx, B * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    fb_invalidate(h);   // copies of the old context lengths say nothing about the new ones
  }
  if (root) CKRT(h, cudaMemcpyAsync(h->ws.root, root, B * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  if (hvec) CKRT(h, cudaMemcpyAsync(h->ws.h, hvec, B * h->dm.d * sizeof(float), cudaMemcpyDeviceToDevice, st));
  h->prefilled = true;
  return RD_OK;
}

int redrafter_set_ctx_bound(rd_handle* h, int32_t max_ctx_now) {
  if (!h || max_ctx_now < 0) return RD_ERR_INVALID_ARG;
  h->ctx_bound = max_ctx_now;
  fb_invalidate(h);
  return RD_OK;
}

int redrafter_profile(rd_handle* h, int enable) {
  if (!h) return RD_ERR_INVALID_ARG;
  h->profiling = enable != 0;
  if (enable)
    for (int c = 0; c < PROF_CLASSES; ++c) { h->ev_used[c] = 0; h->prof_ms[c] = 0; h->prof_bytes[c] = 0; h->prof_n[c] = 0; }
  return RD_OK;
}

int redrafter_profile_read(rd_handle* h, int32_t cls, double* ms, double* bytes, int64_t* launches) {
  if (!h || cls < 0 || cls >= PROF_CLASSES) return RD_ERR_INVALID_ARG;
  double total = h->prof_ms[cls];
  for (size_t i = 0; i + 1 < h->ev_used[cls]; i += 2) {
    CKRT(h, cudaEventSynchronize(h->ev[cls][i + 1]));
    float t = 0.f;
    CKRT(h, cudaEventElapsedTime(&t, h->ev[cls][i], h->ev[cls][i + 1]));
    total += t;
  }
  h->prof_ms[cls] = total;
  h->ev_used[cls] = 0;
  if (ms) *ms = total;
  if (bytes) *bytes = h->prof_bytes[cls];
  if (launches) *launches = h->prof_n[cls];
  return RD_OK;
}

int redrafter_trace(rd_handle* h, int enable, void* stream) {
  if (!h) return RD_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (enable) {
    // minima start at all-ones, maxima at zero
    std::vector<unsigned long long> init((size_t)TRACE_SLOTS * 8);
    for (size_t i = 0; i < init.size(); ++i) init[i] = (i % 8 == 0 || i % 8 == 1 || i % 8 == 3 || i % 8 == 5) ? ~0ull : 0ull;
    CKRT(h, cudaMemcpyAsync(h->ws.trace, init.data(), init.size() * sizeof(unsigned long long), cudaMemcpyHostToDevice, st));
    CKRT(h, cudaStreamSynchronize(st));
    h->trace_next = 0;
    h->trace_bytes.assign(TRACE_SLOTS, 0.0);
    h->trace_prefetch.assign(TRACE_SLOTS, 0.0);
  } else {
    h->trace_next = -1;
  }
  return RD_OK;
}

int redrafter_trace_read(rd_handle* h, void* stream, uint64_t* out, int32_t max_launches) {
  if (!h || !out || max_launches < 0) return RD_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int n = h->trace_next < 0 ? 0 : h->trace_next;
  if (n > max_launches) n = max_launches;
  cudaError_t e = cudaMemcpyAsync(out, h->ws.trace, (size_t)n * 8 * sizeof(unsigned long long), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return -fail(h, RD_ERR_CUDA, "trace read: %s", cudaGetErrorString(e));
  return n;
}

int redrafter_trace_bytes(rd_handle* h, double* out, int32_t max_launches) {
  if (!h || !out || max_launches < 0) return -RD_ERR_INVALID_ARG;
  int n = h->trace_next < 0 ? 0 : h->trace_next;
  if (n > max_launches) n = max_launches;
  for (int i = 0; i < n; ++i) out[i] = i < (int)h->trace_bytes.size() ? h->trace_bytes[i] : 0.0;
  return n;
}

int redrafter_trace_prefetched(rd_handle* h, double* out, int32_t max_launches) {
  if (!h || !out || max_launches < 0) return -RD_ERR_INVALID_ARG;
  int n = h->trace_next < 0 ? 0 : h->trace_next;
  if (n > max_launches) n = max_launches;
  for (int i = 0; i < n; ++i) out[i] = i < (int)h->trace_prefetch.size() ? h->trace_prefetch[i] : 0.0;
  return n;
}

int redrafter_last_packed_rows(rd_handle* h, void* stream, int32_t* n) {
  if (!h || !n) return RD_ERR_INVALID_ARG;
  CKRT(h, cudaMemcpyAsync(n, h->ws.pk.n, (size_t)h->batch * sizeof(int32_t), cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return RD_OK;
}

int redrafter_selftest_wait(rd_handle* h, void* stream) {
  if (!h) return RD_ERR_INVALID_ARG;
  if (!h->chain.ctr) return fail(h, RD_ERR_STATE, "no hand-off counters in this workspace");
  ChainSync cs{h->chain.ctr, h->chain.cum[0] + 0x40000000u, nullptr, h->ws.status, nullptr};
  selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(cs);
  CK(h, cudaGetLastError());
  return RD_OK;
}

int redrafter_poll(rd_handle* h, void* stream) {
  if (!h) return RD_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int32_t v = 0;
  CKRT(h, cudaMemcpyAsync(&v, h->ws.status, sizeof(v), cudaMemcpyDeviceToHost, st));
  CKRT(h, cudaStreamSynchronize(st));
  if (v == 0) return RD_OK;
  CKRT(h, cudaMemsetAsync(h->ws.status, 0, sizeof(int32_t), st));
  if (v & DEV_ERR_TIMEOUT) h->chain_dirty = true;   // launches behind the wait that gave up may not have signalled
  if (v & DEV_ERR_TIMEOUT) return fail(h, RD_ERR_TIMEOUT, "device status 0x%x: a bounded wait gave up", v);
  if (v & DEV_ERR_CAPACITY) return fail(h, RD_ERR_CAPACITY, "device status 0x%x: a KV slot beyond max_ctx was skipped", v);
  return fail(h, RD_ERR_INVALID_ARG, "device status 0x%x: token id or index out of range", v);
}

}  // extern "C"

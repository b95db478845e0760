/*
 * redrafter.h -- C ABI of the B200 (sm_100a) ReDrafter speculative-decode-step library.
 *
 * One step (paper Section 3.4) = draft (Sections 3.1, 3.2) -> pack (Section 3.3,
 * Appendix A.1) -> verify (Section 3.4) -> accept (Section 3.4).
 *
 * Conventions that hold for every call unless a comment says otherwise:
 *   - "device pointer" = CUDA global memory of the current device, owned by the caller;
 *     "host pointer" = ordinary host memory.  The library never frees caller memory.
 *   - Matrices are row-major; a weight of a linear map y = W x is stored [out][in].
 *   - The library allocates NO device memory: all scratch lives in the caller's workspace
 *     given to redrafter_init (size from redrafter_workspace_bytes).
 *   - Calls enqueue work on the given stream and return without synchronising it (the
 *     two exceptions, redrafter_prefill and redrafter_poll, say so).  The calls on one handle
 *     must be issued in stream order on one stream at a time: inside a call consecutive kernels
 *     hand over through counters in the workspace (each is resident before its predecessor has
 *     finished, and waits -- bounded, 1 s -> RD_ERR_TIMEOUT at the next poll -- for the
 *     predecessor's last store), and the bookkeeping of those counters follows the call order.
 *   - Every call returns an rd_status.  Nothing throws, traps or asserts on the device;
 *     problems detected by kernels are recorded in a device status word (redrafter_poll).
 *   - Sizes: B = batch, BW = beam_width, L = beam_length (drafted tokens per candidate =
 *     number of drafter calls, Appendix A.2.1), NMAX = 1 + BW*L packed rows per sequence
 *     (the root token plus every drafted token), MW = ceil(NMAX/32) mask words per row.
 */
#ifndef REDRAFTER_H_
#define REDRAFTER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define RD_API __attribute__((visibility("default")))
#else
#define RD_API
#endif

typedef enum {
  RD_OK = 0,
  RD_ERR_INVALID_ARG = 1, /* null pointer, bad enum value, batch out of range            */
  RD_ERR_SHAPE = 2,       /* unsupported shape (head_dim, alignment, BW > vocab, ...)    */
  RD_ERR_CAPACITY = 3,    /* workspace/KV too small, or the KV cache would overflow      */
  RD_ERR_STATE = 4,       /* call order (e.g. step before prefill)                       */
  RD_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed; see redrafter_last_error */
  RD_ERR_TIMEOUT = 6,     /* a bounded device-side wait gave up                          */
  RD_ERR_UNSUPPORTED = 7
} rd_status;

enum { RD_DTYPE_FP32 = 0, RD_DTYPE_BF16 = 1 };

/* flags for rd_config.flags */
enum {
  RD_FLAG_NO_TREE = 1u << 0,   /* pack without prefix dedup (Figure 3(a)): every candidate keeps its tokens */
  RD_FLAG_FORCE_SIMT = 1u << 1 /* bf16 projections on the CUDA-core path (debug/cross-check)              */
};

/* Model and search shape.  POD; `struct_bytes` must be sizeof(rd_config). */
typedef struct {
  int32_t struct_bytes;
  int32_t n_layers, d_model, n_heads, d_ffn, vocab; /* Llama-style target LLM; head_dim = d_model / n_heads */
  float rms_eps, rope_theta;
  int32_t d_rnn;          /* width of the drafter's RNN state s_t (Section 3.1); must equal d_model         */
  int32_t n_head_layers;  /* residual MLP layers of width d_rnn + d_model in the draft head (Section 3.1)   */
  int32_t dtype;          /* RD_DTYPE_*: storage type of weights, KV cache and projection inputs            */
  int32_t max_batch, max_ctx, beam_width, beam_length;
  uint32_t flags;
} rd_config;

/* Borrowed device pointers to the weights, all in rd_config.dtype.  The per-layer members are
 * HOST arrays (length n_layers / n_head_layers) of device pointers; the arrays are copied by
 * redrafter_init, the weights themselves are only referenced and must outlive the handle. */
typedef struct {
  const void* tok_emb;          /* [vocab][d_model]  input embedding, also the drafter's e_t (Section 3.1) */
  const void* final_norm;       /* [d_model]                                                              */
  const void* lm_head;          /* [vocab][d_model]                                                       */
  const void* const* attn_norm; /* [d_model]                                                              */
  const void* const* wqkv;      /* [3*d_model][d_model]   rows: Q, then K, then V                          */
  const void* const* wo;        /* [d_model][d_model]                                                     */
  const void* const* ffn_norm;  /* [d_model]                                                              */
  const void* const* w_gate_up; /* [2*d_ffn][d_model]     rows: gate, then up                              */
  const void* const* w_down;    /* [d_model][d_ffn]                                                       */
  const void* rnn_u;            /* [d_rnn][d_rnn]    U of s_t = f(U s_{t-1} + W e_t + b) (Section 3.1)     */
  const void* rnn_w;            /* [d_rnn][d_model]  W                                                     */
  const void* rnn_b;            /* [d_rnn]           b                                                     */
  const void* const* head_w;    /* [d_rnn+d_model][d_rnn+d_model]  A_l of x <- x + SiLU(A_l x + c_l)       */
  const void* const* head_b;    /* [d_rnn+d_model]                 c_l                                     */
  const void* draft_out;        /* [vocab][d_rnn+d_model]  projection in front of the drafter's softmax    */
} rd_weights;

/* The packed beam (Section 3.3, Figure 3(b,c)).  All members are device pointers, caller-owned.
 * Rows n >= n[b] are padding with defined values: token 0, pos 0, parent -1, zero mask row. */
typedef struct {
  int32_t* tokens;  /* [B][NMAX]       packed tokens; row 0 is the root (the LLM's guaranteed token)      */
  int32_t* n;       /* [B]             number of packed rows                                              */
  int32_t* unpack;  /* [B][BW][L+1]    packed row holding token j of candidate i (column 0 = root)        */
  int32_t* pos;     /* [B][NMAX]       position id = context length + depth in the tree                   */
  uint32_t* mask;   /* [B][NMAX][MW]   bit m of row n set <=> row n attends packed row m (ancestors+self) */
  int32_t* parent;  /* [B][NMAX]       packed row of the parent node, -1 for the root                     */
} rd_packed;

/* Result of greedy acceptance (Section 3.4).  Device pointers, caller-owned. */
typedef struct {
  int32_t* n_accept; /* [B]       accepted draft tokens a of the best candidate, 0..L                      */
  int32_t* best;     /* [B]       lowest-index candidate with the longest accepted prefix                  */
  int32_t* tokens;   /* [B][L+1]  the a accepted tokens, then the bonus token, then -1 padding             */
} rd_accept_out;

typedef struct rd_handle rd_handle;

/* Bytes of device workspace redrafter_init needs for this config (0 if the config is invalid). */
RD_API size_t redrafter_workspace_bytes(const rd_config* cfg);

/* Bytes of KV cache for this config: [n_layers][2 (K,V)][max_batch][n_heads][max_ctx][head_dim] of dtype.
 * K is stored after the rotary embedding. */
RD_API size_t redrafter_kv_bytes(const rd_config* cfg);

/* Create a handle.  `kv_cache` and `workspace` are device pointers (256-byte aligned) that the
 * handle uses until redrafter_destroy; their contents are owned by the library while it lives.
 * Host-only apart from building TMA descriptors; enqueues a clear of the state on `stream 0` and, in bf16 with head
 * dimension 128, clears the KV cache (the tensor-core attention kernel multiplies the value rows of masked-out keys by
 * exact zeros, so every slot has to hold finite values).
 * Errors: INVALID_ARG, SHAPE (head_dim not 64 or 128, d_model/d_ffn not multiples of 64 in bf16,
 * beam_width > vocab, NMAX > 1024), CAPACITY (buffers too small), CUDA. */
RD_API int redrafter_init(const rd_config* cfg, const rd_weights* weights, void* kv_cache, size_t kv_bytes,
                   void* workspace, size_t ws_bytes, rd_handle** out);

/* Free the host-side handle.  Does not touch device memory. */
RD_API int redrafter_destroy(rd_handle* h);

/* Message of the last failing call on this handle (host string, valid until the next call).
 * With h == NULL: why the last redrafter_init failed. */
RD_API const char* redrafter_last_error(const rd_handle* h);

/* Causal forward over the prompts (the state before the first step, Figure 2): fills the KV
 * cache, sets ctx[b] = prompt_len[b], root g[b] = the LLM's greedy token after the prompt and
 * h[b] = its last hidden state (after the final norm).
 * tokens: HOST pointer [batch][max_prompt] (row stride max_prompt); prompt_len: HOST [batch].
 * Copies the inputs from pageable host memory, so it may block the host; the forward itself is
 * only enqueued.  Errors: INVALID_ARG, CAPACITY (prompt_len + NMAX > max_ctx). */
RD_API int redrafter_prefill(rd_handle* h, const int32_t* tokens, const int32_t* prompt_len, int32_t max_prompt,
                      int32_t batch, void* stream);

/* Beam search over the RNN drafter (Sections 3.1, 3.2) from the current state (g, h).
 * beams: device [B][BW][L] int32, candidates sorted by cumulative log-probability (descending,
 * ties by flat candidate index); scores: device [B][BW] fp32 natural-log probabilities. */
RD_API int redrafter_draft(rd_handle* h, void* stream, int32_t* beams, float* scores);

/* Dynamic tree attention packing (Section 3.3, Appendix A.1) of `beams` (device [B][BW][L]) under
 * the current roots and context lengths into `out` (see rd_packed). */
RD_API int redrafter_pack(rd_handle* h, const int32_t* beams, void* stream, const rd_packed* out);

/* Target-LLM forward over the packed rows against the KV cache and the tree mask (Section 3.4).
 * K/V of row n are written provisionally to cache slot ctx[b] + n.
 * argmax: device [B][NMAX] int32 the LLM's next token per packed row: greedy (lowest id on ties), or drawn
 *   after redrafter_set_sampling; -1 on padding;
 * hidden: device [B][NMAX][d_model] fp32 output of the final norm, or NULL;
 * logits: device [B][NMAX][vocab] fp32, or NULL.  Padding rows are left untouched in hidden/logits. */
RD_API int redrafter_verify(rd_handle* h, const rd_packed* packed, void* stream, int32_t* argmax, float* hidden,
                     float* logits);

/* Greedy acceptance (token matches, Section 3.4) + KV-cache compaction + hand-off of the bonus
 * token and its hidden state to the next step.  `hidden` is the buffer redrafter_verify filled
 * (must not be NULL).  Advances ctx[b] by 1 + n_accept[b].  `out` members may each be NULL. */
RD_API int redrafter_accept(rd_handle* h, const int32_t* beams, const rd_packed* packed, const int32_t* argmax,
                     const float* hidden, void* stream, const rd_accept_out* out);

/* redrafter_accept for callers that cannot provide scratch memory.  (The paper has no counterpart: this
 * is a deployment variant of the accept step above, same inputs, same results.)
 *
 * Who needs it: code that runs where device allocation is off the table -- inside a latency-critical
 * serving loop that must never enter the allocator, in a plugin whose host owns all GPU memory and
 * hands out none, or after start-up in a process that has given its whole memory budget away.  Such a
 * caller can still drive the accept step: the three per-sequence temporaries that the accept and the
 * KV-compaction kernels pass to each other live in a fixed array inside the library instead of in
 * memory the caller supplies.  This call performs no cudaMalloc/cudaFree and uses no allocating
 * library routine.
 *
 * Limits and rules:
 *  - at most 4096 sequences per call (RD_ERR_CAPACITY beyond that, nothing is enqueued); the array
 *    takes 48 KB on every GPU that loads the library, until the process exits;
 *  - the first call on each device looks up the array's device address (one runtime query, with that
 *    device current) and remembers it: make that first call outside any stream capture;
 *  - all calls on a device share the one array and it keeps the last call's values.  Nothing in it has
 *    to start at zero (every entry that is read is written first by the same call), but two calls
 *    whose kernels overlap on the GPU -- different streams, no ordering between them -- race on it:
 *    order them.  redrafter_accept has no such restriction across handles.
 * Everything else (arguments, outputs, state update, errors) is exactly as for redrafter_accept. */
RD_API int redrafter_accept_static(rd_handle* h, const int32_t* beams, const rd_packed* packed, const int32_t* argmax,
                                   const float* hidden, void* stream, const rd_accept_out* out);

/* The whole step in one call, using workspace-internal intermediates.  With planted_beams
 * (device [B][BW][L]) non-NULL the drafter still runs but the planted candidates are packed and
 * verified.  `out` may be NULL.  Errors: STATE (no prefill yet), CAPACITY (host-tracked upper bound
 * of the context + NMAX exceeds max_ctx; nothing is enqueued). */
RD_API int redrafter_step(rd_handle* h, const int32_t* planted_beams, void* stream, const rd_accept_out* out);

/* Plain autoregressive step built from the same kernels (the comparator of every speedup in
 * Section 4): feeds g at position ctx, advances ctx by 1, sets the new g and h.
 * token: device [B] int32 (the new g), may be NULL. */
RD_API int redrafter_ar_step(rd_handle* h, void* stream, int32_t* token);

/* Acceptance at temperature > 0 (Section 3.4 names rejection sampling as the other end of the selection
 * methods and gives no procedure).  Beam search proposes tokens deterministically, so the proposal at a tree
 * node is a point mass per child; the accept/resample rule of speculative sampling then has the law of
 * "draw y from the LLM's distribution p at the node and descend iff y is a child".  After this call every
 * token the LLM chooses -- the root after the prompt, the per-row tokens of redrafter_verify (its `argmax`
 * output) and redrafter_step, the token of redrafter_ar_step -- is such a draw from softmax(logits / T),
 * made by the Gumbel-max rule: argmax_v (logit_v / T - ln(-ln u_v)), lowest id on ties, with
 * u_v = (top 23 bits of word (v mod 4) of Philox-4x32-10(counter = (v / 4, position, sequence, 0),
 * key = (seed mod 2^32, seed >> 32)) + 1/2) / 2^23 and `position` the index of the token being chosen in
 * its sequence (prompt tokens count from 0), `sequence` its batch index.  The draw for a position therefore
 * does not depend on the branch, the row or the step that reaches it: speculative steps and
 * redrafter_ar_step generate the same tokens.  Acceptance, compaction and hand-off are unchanged (they
 * compare tokens).  temperature == 0 restores greedy choice (the default).  Takes effect for calls made
 * after it; enqueues nothing.  Errors: INVALID_ARG (negative or non-finite temperature). */
RD_API int redrafter_set_sampling(rd_handle* h, float temperature, uint64_t seed);

/* Copy the decode state out of / into the handle.  Device pointers; any may be NULL.
 * ctx [B] int32 context lengths, root [B] int32 guaranteed tokens, hvec [B][d_model] fp32. */
RD_API int redrafter_get_state(rd_handle* h, void* stream, int32_t* ctx, int32_t* root, float* hvec);
RD_API int redrafter_set_state(rd_handle* h, void* stream, const int32_t* ctx, const int32_t* root, const float* hvec,
                        int32_t batch);

/* Tell the handle the largest context length any sequence can have now.  The handle keeps this bound on the host
 * (it never reads device memory synchronously): the capacity check (RD_ERR_CAPACITY when bound + 1 + beam_width *
 * beam_length > max_ctx) and the attention launch geometry follow it.  Every step adds 1 + beam_length to it, the most
 * a step can accept; every eighth call also enqueues a copy of the true context lengths to pinned host memory, and a
 * later call that finds the copy complete lowers the bound to what it implies, so the bound runs ahead of the real
 * contexts by at most eight steps' worth.  A caller that passes `ctx` to redrafter_set_state MUST call this function
 * too (set_state does not read the array it is given): the bound is not raised by the feedback. */
RD_API int redrafter_set_ctx_bound(rd_handle* h, int32_t max_ctx_now);

/* Synchronise `stream`, read the device status word and clear it.  Returns RD_OK or the first
 * error a kernel recorded (e.g. an out-of-range token id was skipped). */
RD_API int redrafter_poll(rd_handle* h, void* stream);

/* Per-launch device timing, for measurement only (off by default).  While enabled, every launch of
 * redrafter_step is bracketed by CUDA events on its stream, summed by class: 0 projections,
 * 1 attention, 2 RMSNorm, 3 rotary + KV write, 4 SwiGLU, 5 drafter selection kernels, 6 pack/accept,
 * 7 the rest.  The events are created on first use.  redrafter_profile(h, 1) also clears the totals.
 * redrafter_profile_read waits for the recorded events and returns, for one class, the summed
 * device time in ms, the summed algorithmic weight bytes of the launches (class 0 only: N*K*element
 * size per projection) and the number of launches.  Outputs are HOST pointers, each may be NULL.
 * The event pool grows with the launches between reads: read at least once per step. */
RD_API int redrafter_profile(rd_handle* h, int enable);
RD_API int redrafter_profile_read(rd_handle* h, int32_t cls, double* ms, double* bytes, int64_t* launches);

/* In-kernel timeline, for measurement only.  After redrafter_trace(h, 1, stream) the next launches of
 * the traced kernels (up to 512, in launch order) each record eight %globaltimer values in ns
 * (fields a kernel does not write keep their initial value: all ones in [0], [1], [3], [5], zero elsewhere):
 *   tensor-core projection: [0] first CTA entered, [1]/[2] first/last producer past its dependency wait,
 *                           [3]/[4] first/last MMA issuer done, [5]/[6] first/last CTA done, [7] last producer
 *                           ready to wait (its first ring of weight tiles requested);
 *   short kernels of the chained loops (RMSNorm, rotary, SwiGLU, drafter activation, selection segments):
 *                           [0]/[7] first/last CTA entered, [1]/[2] first/last CTA past its wait,
 *                           [5]/[6] first/last CTA done;
 *   tensor-core attention:  [0] entered, [1] past its wait, [2] Q loaded, [3] key chunks done (the CTA of head 0,
 *                           sequence 0, split 0); [6] last CTA done;
 *   selection, two-kernel form (its second kernel): [0] first CTA entered, [1] first past the wait, [2] last CTA's
 *                           rows merged, [6] last CTA done;  single-kernel form (last CTA): [0] entered, [1] past
 *                           the wait, [2] logits in shared memory, [3] threshold found, [4] row ranked,
 *                           [5] arrival counted, [6] pruning done.
 * redrafter_trace_read synchronises the stream, copies the records of the launches traced so far to
 * the HOST buffer out[max_launches][8] and returns their number (or a negative rd_status).
 * redrafter_trace_bytes fills the HOST buffer out[max_launches] with the weight bytes (N*K*element size) of each of
 * those launches, 0 for the ones that are not projections, and returns the same number. */
RD_API int redrafter_trace(rd_handle* h, int enable, void* stream);
RD_API int redrafter_trace_read(rd_handle* h, void* stream, uint64_t* out, int32_t max_launches);
RD_API int redrafter_trace_bytes(rd_handle* h, double* out, int32_t max_launches);
/* Same layout: of those weight bytes, the ones each projection launch requests BEFORE its dependency wait (the first
 * ring-full of stages of every CTA, which stream in under the preceding kernel).  A rate "in place" divides the
 * remaining bytes by the time after the wait. */
RD_API int redrafter_trace_prefetched(rd_handle* h, double* out, int32_t max_launches);

/* Self-test of the bounded device-side waits (the paper has no counterpart).  Enqueues one tiny kernel that waits on
 * a hand-off counter value that nothing will ever produce: the wait gives up after its limit (about one second) and
 * records it, the kernel returns, the context stays usable; the next redrafter_poll returns RD_ERR_TIMEOUT and clears
 * the status word.  Nothing else of the handle's state is touched. */
RD_API int redrafter_selftest_wait(rd_handle* h, void* stream);

/* Number of kernels this handle has launched since it was created (for launch accounting). */
RD_API int64_t redrafter_launch_count(const rd_handle* h);

/* Packed rows N_b (root + deduplicated draft tokens, Section 3.3) of every sequence in the most recent redrafter_step:
 * copies n[batch] int32 to the DEVICE buffer `n`, enqueued on `stream`.  The measure of what dynamic tree attention
 * saves: without it a step verifies 1 + beam_width * beam_length rows per sequence (Figure 5, left). */
RD_API int redrafter_last_packed_rows(rd_handle* h, void* stream, int32_t* n);

/* Diagnostic (the paper has no counterpart): copies rows [0, rows) of the logits computed by the handle's last
 * forward pass into the DEVICE buffer out[rows][vocab] (fp32), enqueued on `stream`.  After redrafter_ar_step row b
 * is sequence b's next-token logits; after redrafter_verify / redrafter_step the rows are the packed rows of all
 * sequences back to back.  rows must not exceed max_batch * (1 + beam_width * beam_length): RD_ERR_INVALID_ARG. */
RD_API int redrafter_last_logits(rd_handle* h, void* stream, float* out, int32_t rows);

/* Which kernel variants the handle's attention and projection launches have taken since it was created (the paper
 * has no counterpart: Section 3.4's verification pass is one attention over the cache plus the tree mask, and this
 * library picks among several kernels for it by row count and context length).  Fills the HOST array out[0 .. n-1],
 * n <= RD_ROUTE_COUNT, with launch counts; tests use it to check that a workload exercises the kernel it is meant
 * to.  Never touches the device. */
enum {
  RD_ROUTE_ATT_ROWS16 = 0,        /* 16-row tiles, four-chunk ring (decode steps) */
  RD_ROUTE_ATT_ROWS16_SHALLOW = 1,/* 16-row tiles, two-chunk ring (more tiles than SMs) */
  RD_ROUTE_ATT_ROWS64 = 2,        /* 64-row tiles */
  RD_ROUTE_ATT_ROWS128_TC5 = 3,   /* 128-row tiles on tcgen05 */
  RD_ROUTE_ATT_KEY_SPLIT = 4,     /* of the 16-row launches: those whose keys were split over several CTAs */
  RD_ROUTE_ATT_FP32 = 5,          /* the fp32 configuration's kernel */
  RD_ROUTE_GEMM_PAIRS = 6,        /* projections on CTA pairs */
  RD_ROUTE_GEMM_ONE_CTA = 7,      /* projections on single CTAs (tensor cores) */
  RD_ROUTE_GEMM_SIMT = 8,         /* projections on CUDA cores */
  RD_ROUTE_COUNT = 9
};
RD_API int redrafter_route_counts(const rd_handle* h, int64_t* out, int32_t n);

#ifdef __cplusplus
}
#endif
#endif /* REDRAFTER_H_ */

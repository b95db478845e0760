"""CPU oracle for one ReDrafter speculative decode step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain reference that the CUDA
library is compared against.  It shares no code with the CUDA path and must never
be imported by the product package; only tests, the smoke check and the benchmark's
CPU-baseline leg use it.

Everything is numpy, float64 by default, one sequence at a time (a batch is a
Python loop over independent sequences, Appendix A.1: the batch is only a leading
dimension).  The steps follow the paper's order (Section 3.4):

    draft (Sections 3.1, 3.2)  ->  dedup_prefix / pack_beam (Section 3.3, Appendix A.1)
    ->  LLM verification forward (Section 3.4)  ->  greedy acceptance (Section 3.4)

The paper is silent on several points (activation, head depth, the LLM's
architecture, KV cache handling, tie breaking).  The readings used here:

  * f = SiLU; the head is `n_head_layers` residual layers x <- x + SiLU(A x + c) of
    width 2d followed by a bias-free projection to the vocabulary and a softmax.
  * s_1 := e_1 is the embedding of the token the LLM just produced (Section 3.1);
    the first drafter call applies the head to [s_1, h] directly, later calls
    first update s_t = f(U s_{t-1} + W e_t + b) with e_t the embedding of the token
    drafted by the previous call.
  * Beam length L = number of drafter calls = drafted tokens per candidate
    (Appendix A.2.1); the guaranteed root token is extra.
  * The LLM is Llama-style: pre-norm RMSNorm, rotary embedding with the half-split
    pairing (i, i + hd/2), multi-head attention with scale hd^-1/2, SwiGLU, no biases.
  * Candidates are ordered by (score descending, flat index ascending); argmax ties
    go to the lowest index; equal accepted lengths go to the lowest beam index.
  * The dedup listing in Appendix A.1 is read through its comment and its printed
    example: compare candidate i with candidate j position by position, a prefix of
    length j+1 is shared when all of its j+1 positions match, and the FIRST such
    candidate is reported.

  * Acceptance at temperature > 0 (Section 3.4 names rejection sampling and gives no
    procedure).  Beam search proposes tokens deterministically, so the proposal at a
    tree node is a point mass per child.  For such a proposal the accept/resample
    rule of speculative sampling -- keep the proposed token x with probability
    min(1, p(x)/q(x)) = p(x), otherwise draw from the residual, which is p with x
    removed, child after child -- has the same law as: draw y ~ p at the node and
    descend iff y is one of its children.  The draw is made with the Gumbel-max rule
    y = argmax_v (logit_v / T + G_v), G_v = -ln(-ln u_v), with u_v from the
    counter-based generator Philox-4x32-10 keyed by (seed; sequence, position of the
    token being chosen, v), so the token chosen for a position does not depend on the
    branch or the step that reaches it: speculative decoding reproduces plain sampled
    decoding token for token.

  * Precision (the paper states none).  By default everything is computed in the
    working precision.  The bf16 configurations of the CUDA library STORE some
    intermediates in bfloat16: every vector that feeds a projection (the normalised
    residual stream, the attention output, the SwiGLU output, the drafter's [s, e] and
    [s, h] vectors and its head activations), the rotated queries and keys and the values
    (the K/V cache), and the softmax weights that multiply V.  With store="bf16" the
    functions below round exactly those arrays, element by element, to the nearest
    bfloat16 (ties to even) and change nothing else: no blocking, no reordering, sums
    and softmax statistics stay in the working precision, the residual stream and the
    hidden state handed to the drafter stay unrounded.  Comparing the two modes on the
    CPU measures what that storage costs in accuracy, independently of any kernel.

Parity pins (tests/test_oracle_*.py): the printed dedup example, brute-force
prefix sets, packed-tree == per-beam causal verification, speculative == plain
greedy decoding, beam width 1 == greedy drafting, exhaustive beam search on a tiny
vocabulary, closed forms for the RNN cell and the head, library cross-checks; for
sampling: the generator's published known answers, sample frequencies against the
softmax, the accept/resample rule worked out exactly on small cases, speculative ==
plain sampled decoding; for store="bf16": round_bf16 against the bit-level definition
and a library cast, idempotence, the unrounded mode's own pins re-run in this mode
(packed-tree == per-beam, speculative == plain decoding, beam width 1 == greedy
drafting, scores == sequence log-probabilities), and the size of the storage error and
its growth with depth (tests/test_oracle_storage.py).
Parity unpinned: nothing in the paper prints a weights-to-beams example, so the
drafter's exact beams are pinned by properties only.
"""
from __future__ import annotations

import numpy as np

F = np.float64


# ----------------------------------------------------------------------------
# elementary functions
# ----------------------------------------------------------------------------
def _c(a, dtype):
    """The array in the working precision (no copy when it already is)."""
    return np.asarray(a, dtype=dtype)


def convert_weights(W, D, dtype):
    """Copies of the weight dicts in the working precision, so later calls do not convert again."""
    def conv(v):
        return [_c(t, dtype) for t in v] if isinstance(v, list) else _c(v, dtype)
    return {k: conv(v) for k, v in W.items()}, {k: conv(v) for k, v in D.items()}


def round_bf16(a):
    """Every element rounded to the nearest bfloat16 (8 significand bits, float32's exponent range; ties to even),
    returned in the input's dtype.  The value is first taken to float32, as the stored intermediates are."""
    a = np.asarray(a)
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)                 # last bit that survives: decides ties
    u = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return u.view(np.float32).astype(a.dtype if a.dtype.kind == "f" else np.float32)


def _st(a, store):
    """`a` as it is stored between two operations: unchanged, or rounded to bfloat16."""
    if store is None:
        return a
    assert store == "bf16"
    return round_bf16(a)


def silu(x):
    return x / (1.0 + np.exp(-x))


def log_softmax(z):
    """Natural-log softmax of a vector (Section 3.1: standard softmax layer)."""
    m = np.max(z)
    return z - (m + np.log(np.sum(np.exp(z - m))))


def rmsnorm(x, gain, eps):
    """x: [rows, d].  y = x / sqrt(mean(x^2) + eps) * gain."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(x, pos, theta):
    """Rotary embedding, half-split pairing.  x: [rows, heads, hd]; pos: [rows]."""
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = theta ** (-(np.arange(half, dtype=F) * 2.0) / hd)
    ang = np.asarray(pos, dtype=F)[:, None] * inv_freq[None, :]          # [rows, half]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    x1 = x[..., :half]
    x2 = x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def argmax_first(v):
    """Index of the maximum; the lowest index on ties."""
    return int(np.argmax(v))


def top_k_ordered(values, k):
    """Indices of the k largest values ordered by (value desc, index asc)."""
    order = np.lexsort((np.arange(values.shape[0]), -values))
    return order[:k]


# ----------------------------------------------------------------------------
# token choice at temperature > 0 (Section 3.4: "rejection sampling")
# ----------------------------------------------------------------------------
PHILOX_M0, PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
PHILOX_W0, PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32(counter, key, rounds=10):
    """Philox-4x32 (Salmon et al., SC'11): four 32-bit counter words, two key words.

    counter: four integers or equally shaped integer arrays; key: two integers.
    Returns four uint64 arrays holding 32-bit values.
    """
    c = [np.asarray(x, dtype=np.uint64) & np.uint64(0xFFFFFFFF) for x in counter]
    c = list(np.broadcast_arrays(*c))
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    lo32, sh = np.uint64(0xFFFFFFFF), np.uint64(32)
    for _ in range(rounds):
        p0 = np.uint64(PHILOX_M0) * c[0]        # 32 x 32 -> 64 bits, exact in uint64
        p1 = np.uint64(PHILOX_M1) * c[2]
        c = [(p1 >> sh) ^ c[1] ^ np.uint64(k0), p1 & lo32, (p0 >> sh) ^ c[3] ^ np.uint64(k1), p0 & lo32]
        k0 = (k0 + PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + PHILOX_W1) & 0xFFFFFFFF
    return c


def uniform_open(x32):
    """32 random bits -> u in (0, 1): the top 23 bits plus one half, over 2^23 (exact in fp32 and fp64)."""
    return ((np.asarray(x32, dtype=np.uint64) >> np.uint64(9)).astype(np.float64) + 0.5) / float(1 << 23)


def gumbel_noise(seed, seq, pos, vocab):
    """G_v = -ln(-ln u_v), v < vocab, for the token at position `pos` of sequence `seq`.

    Vocabulary entries 4k .. 4k+3 are the four output words of the counter (k, pos, seq, 0)
    under the key (seed mod 2^32, seed >> 32).
    """
    blocks = np.arange((vocab + 3) // 4, dtype=np.uint64)
    words = philox4x32((blocks, pos, seq, 0), (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))
    u = uniform_open(np.stack(words, axis=1).reshape(-1)[:vocab])
    return -np.log(-np.log(u))


def choose_token(logits, sampling=None, seq=0, pos=0, want_scores=False):
    """The LLM's token for position `pos` given its logits there.

    sampling None (or temperature 0): the greedy token.  Otherwise sampling =
    dict(temperature=T, seed=s): a draw from softmax(logits / T) by the Gumbel-max rule.
    """
    z = np.asarray(logits, dtype=F)
    if sampling is not None and sampling["temperature"] > 0:
        z = z / sampling["temperature"] + gumbel_noise(sampling["seed"], seq, pos, z.shape[0])
    return (argmax_first(z), z) if want_scores else argmax_first(z)


def choose_rows(logits, pos, sampling=None, seq=0):
    """choose_token for every row; row r's logits choose the token at position pos[r] + 1."""
    return np.array([choose_token(logits[r], sampling, seq, int(pos[r]) + 1) for r in range(logits.shape[0])], dtype=np.int64)


# ----------------------------------------------------------------------------
# target LLM (verification forward, Section 3.4)
# ----------------------------------------------------------------------------
class KVCache:
    """Per-sequence cache: k, v of shape [n_layers, max_ctx, n_heads, hd]."""

    def __init__(self, n_layers, max_ctx, n_heads, hd, dtype=F):
        self.k = np.zeros((n_layers, max_ctx, n_heads, hd), dtype=dtype)
        self.v = np.zeros((n_layers, max_ctx, n_heads, hd), dtype=dtype)


def llm_forward(W, cfg, tokens, pos, mask, kv, ctx, dtype=F, want_logits=True, store=None):
    """Forward over `tokens` (rows) with explicit positions and mask.

    Row n attends cache slots [0, ctx) and the rows m with mask[n, m] True (self
    included); its key/value are written provisionally to slot ctx + n.
    Returns (hidden [rows, d] after the final norm, logits [rows, V] or None).
    store="bf16": projection inputs, Q, K, V and the softmax weights are rounded (module docstring).
    """
    H = cfg["n_heads"]
    d = cfg["d_model"]
    hd = d // H
    eps = cfg["rms_eps"]
    theta = cfg["rope_theta"]
    tokens = np.asarray(tokens)
    n = tokens.shape[0]
    assert ctx + n <= kv.k.shape[1], "KV cache capacity exceeded"
    mask = np.asarray(mask, dtype=bool)
    x = np.asarray(W["tok_emb"][tokens], dtype=dtype)
    scale = 1.0 / np.sqrt(hd)
    for l in range(cfg["n_layers"]):
        a = _st(rmsnorm(x, _c(W["attn_norm"][l], dtype), eps), store)
        qkv = a @ _c(W["wqkv"][l], dtype).T                          # [n, 3d]
        q = _st(rope(qkv[:, :d].reshape(n, H, hd), pos, theta), store)
        k = _st(rope(qkv[:, d:2 * d].reshape(n, H, hd), pos, theta), store)
        v = _st(qkv[:, 2 * d:].reshape(n, H, hd), store)
        kv.k[l, ctx:ctx + n] = k
        kv.v[l, ctx:ctx + n] = v
        attn = np.zeros((n, H, hd), dtype=dtype)
        for r in range(n):
            slots = np.concatenate([np.arange(ctx), ctx + np.nonzero(mask[r])[0]])
            kk = kv.k[l, slots].astype(dtype)                           # [keys, H, hd]
            vv = kv.v[l, slots].astype(dtype)
            sc = np.einsum("hd,khd->hk", q[r], kk) * scale              # [H, keys]
            sc = sc - sc.max(axis=1, keepdims=True)
            p = np.exp(sc)
            # softmax(sc) V as (p V) / sum(p): the stored copy of p multiplies V, the sum is exact
            attn[r] = np.einsum("hk,khd->hd", _st(p, store), vv) / p.sum(axis=1, keepdims=True)
        x = x + _st(attn.reshape(n, d), store) @ _c(W["wo"][l], dtype).T
        f = _st(rmsnorm(x, _c(W["ffn_norm"][l], dtype), eps), store)
        gu = f @ _c(W["w_gate_up"][l], dtype).T                      # [n, 2F]: gate rows then up rows
        Fd = cfg["d_ffn"]
        act = _st(silu(gu[:, :Fd]) * gu[:, Fd:], store)
        x = x + act @ _c(W["w_down"][l], dtype).T
    hidden = rmsnorm(x, _c(W["final_norm"], dtype), eps)
    logits = _st(hidden, store) @ _c(W["lm_head"], dtype).T if want_logits else None
    return hidden, logits


def prefill(W, cfg, prompt, kv, dtype=F, sampling=None, seq=0, store=None):
    """Causal forward over the prompt.  Returns (ctx, root token g, h)."""
    P = len(prompt)
    mask = np.tril(np.ones((P, P), dtype=bool))
    hidden, _ = llm_forward(W, cfg, prompt, np.arange(P), mask, kv, 0, dtype, want_logits=False, store=store)
    logits_last = _st(hidden[P - 1], store) @ _c(W["lm_head"], dtype).T
    return P, choose_token(logits_last, sampling, seq, P), hidden[P - 1].copy()


def ar_step(W, cfg, kv, ctx, g, dtype=F, sampling=None, seq=0, store=None):
    """One plain autoregressive step: feed g at position ctx, return next token, h, logits."""
    hidden, logits = llm_forward(W, cfg, [g], [ctx], np.ones((1, 1), bool), kv, ctx, dtype, store=store)
    return choose_token(logits[0], sampling, seq, ctx + 1), hidden[0].copy(), logits[0]


# ----------------------------------------------------------------------------
# drafter (Sections 3.1 and 3.2)
# ----------------------------------------------------------------------------
def rnn_cell(D, s_prev, e, dtype=F, store=None):
    """s_t = f(U s_{t-1} + W e_t + b) (Section 3.1)."""
    return silu(_c(D["rnn_u"], dtype) @ _st(s_prev, store) + _c(D["rnn_w"], dtype) @ _st(e, store) + _c(D["rnn_b"], dtype))


def draft_head(D, g_t, dtype=F, store=None):
    """MLP layers with skip connections, then the vocabulary projection (Section 3.1).  Returns logits.
    store="bf16": each projection reads a rounded copy of x; the skip path keeps x itself."""
    x = g_t
    for A, c in zip(D["head_w"], D["head_b"]):
        x = x + silu(_c(A, dtype) @ _st(x, store) + _c(c, dtype))
    return _c(D["draft_out"], dtype) @ _st(x, store)


def beam_search(D, E, g, h, beam_width, beam_length, dtype=F, return_logp=False, store=None):
    """Beam search over the drafter (Section 3.2).

    Returns beams [BW, L] (int64), scores [BW]: candidates sorted by cumulative
    log-probability, descending.  With return_logp also the per-call candidate
    arrays (for gap-gated comparisons).
    """
    V = D["draft_out"].shape[0]
    assert beam_width <= V
    E = _c(E, dtype)
    h = np.asarray(h, dtype=dtype)
    s1 = E[g]
    logp = log_softmax(draft_head(D, np.concatenate([s1, h]), dtype, store))
    top = top_k_ordered(logp, beam_width)
    hist = [[int(v)] for v in top]
    scores = logp[top].copy()
    states = [s1.copy() for _ in range(beam_width)]
    cand_log = [logp.copy()]
    for _t in range(2, beam_length + 1):
        cand = np.empty(beam_width * V, dtype=dtype)
        new_states = []
        for b in range(beam_width):
            s = rnn_cell(D, states[b], E[hist[b][-1]], dtype, store)
            new_states.append(s)
            lp = log_softmax(draft_head(D, np.concatenate([s, h]), dtype, store))
            cand[b * V:(b + 1) * V] = scores[b] + lp
        top = top_k_ordered(cand, beam_width)
        cand_log.append(cand)
        hist = [hist[int(c) // V] + [int(c) % V] for c in top]
        states = [new_states[int(c) // V] for c in top]
        scores = cand[top].copy()
    beams = np.array(hist, dtype=np.int64).reshape(beam_width, beam_length)
    if return_logp:
        return beams, scores, cand_log
    return beams, scores


def sequence_logprob(D, E, g, h, seq, dtype=F, store=None):
    """log p_draft(seq | g, h): the drafter run along one fixed sequence."""
    E = _c(E, dtype)
    s = E[g]
    total = 0.0
    for t, tok in enumerate(seq):
        if t > 0:
            s = rnn_cell(D, s, E[seq[t - 1]], dtype, store)
        lp = log_softmax(draft_head(D, np.concatenate([s, np.asarray(h, dtype=dtype)]), dtype, store))
        total += lp[tok]
    return total


# ----------------------------------------------------------------------------
# dynamic tree attention (Section 3.3, Appendix A.1)
# ----------------------------------------------------------------------------
def dedup_prefix(beam):
    """prefix_tree[i][j] = smallest k with beam[k][:j+1] == beam[i][:j+1]."""
    # The definition written out (Appendix A.1, first paragraph): for every candidate
    # i and prefix length j+1, scan the candidates in index order and report the
    # first one whose leading j+1 tokens are the same.
    beam = np.asarray(beam)
    bw, bl = beam.shape
    prefix_tree = np.zeros((bw, bl), dtype=np.int64)
    for i in range(bw):
        for j in range(bl):
            for k in range(bw):
                if all(beam[k][c] == beam[i][c] for c in range(j + 1)):
                    prefix_tree[i, j] = k
                    break
    return prefix_tree


def pack_beam(beam_aug, ctx):
    """Compress the augmented beam [root | drafts] ([BW, L+1]) into the packed beam.

    Token (i, j) is kept iff prefix_tree[i][j] == i (Appendix A.1: tokens with
    prefix_tree[i][j] < i can be condensed); kept tokens are numbered in row-major
    order.  Returns a dict with
      tokens[N], n, unpack[BW, L+1], pos[N] = ctx + depth, depth[N], parent[N]
      (-1 for the root), mask[N, N] (row n sees its ancestors and itself).
    """
    beam_aug = np.asarray(beam_aug)
    bw, cols = beam_aug.shape
    assert np.all(beam_aug[:, 0] == beam_aug[0, 0]), "column 0 is the shared root"
    pt = dedup_prefix(beam_aug)
    keep = pt == np.arange(bw)[:, None]
    index = np.cumsum(keep.reshape(-1)).reshape(bw, cols) - 1            # inclusive scan - 1 on kept
    n = int(keep.sum())
    tokens = np.zeros(n, dtype=np.int64)
    depth = np.zeros(n, dtype=np.int64)
    unpack = np.zeros((bw, cols), dtype=np.int64)
    for i in range(bw):
        for j in range(cols):
            unpack[i, j] = index[pt[i, j], j]
            if keep[i, j]:
                tokens[index[i, j]] = beam_aug[i, j]
                depth[index[i, j]] = j
    parent = np.full(n, -1, dtype=np.int64)
    mask = np.zeros((n, n), dtype=bool)
    for i in range(bw):
        for j in range(cols):
            r = unpack[i, j]
            if j > 0:
                parent[r] = unpack[i, j - 1]
            mask[r, unpack[i, :j + 1]] = True
    return dict(tokens=tokens, n=n, unpack=unpack, pos=ctx + depth, depth=depth,
                parent=parent, mask=mask, prefix_tree=pt)


def flat_beam(beam_aug, ctx):
    """The no-tree-attention arm (Figure 3(a)): every candidate keeps all its tokens
    except the shared root, which is sent once.  Same output dict as pack_beam."""
    beam_aug = np.asarray(beam_aug)
    bw, cols = beam_aug.shape
    n = 1 + bw * (cols - 1)
    tokens = np.zeros(n, dtype=np.int64)
    depth = np.zeros(n, dtype=np.int64)
    unpack = np.zeros((bw, cols), dtype=np.int64)
    tokens[0] = beam_aug[0, 0]
    for i in range(bw):
        for j in range(1, cols):
            r = 1 + i * (cols - 1) + (j - 1)
            unpack[i, j] = r
            tokens[r] = beam_aug[i, j]
            depth[r] = j
    parent = np.full(n, -1, dtype=np.int64)
    mask = np.zeros((n, n), dtype=bool)
    for i in range(bw):
        for j in range(cols):
            r = unpack[i, j]
            if j > 0:
                parent[r] = unpack[i, j - 1]
            mask[r, unpack[i, :j + 1]] = True
    return dict(tokens=tokens, n=n, unpack=unpack, pos=ctx + depth, depth=depth,
                parent=parent, mask=mask)


# ----------------------------------------------------------------------------
# acceptance + KV compaction (Section 3.4)
# ----------------------------------------------------------------------------
def accept_greedy(beams, unpack, llm_argmax):
    """Longest prefix of a candidate whose tokens equal the LLM's own tokens.

    beams [BW, L]; unpack [BW, L+1] (column 0 = root); llm_argmax[N] = the LLM's
    next token after each packed node (greedy, or drawn: see choose_token).  Returns (a, best, emitted) where
    emitted = accepted draft tokens followed by the bonus token.
    """
    beams = np.asarray(beams)
    bw, L = beams.shape
    best, a = 0, -1
    for i in range(bw):
        ai = 0
        while ai < L and beams[i, ai] == llm_argmax[unpack[i, ai]]:
            ai += 1
        if ai > a:
            a, best = ai, i
    bonus = int(llm_argmax[unpack[best, a]])
    emitted = [int(t) for t in beams[best, :a]] + [bonus]
    return a, best, emitted


def compact_kv(kv, ctx, unpack, best, a):
    """Move the accepted path's provisional K/V rows to slots ctx+1 .. ctx+a."""
    for j in range(1, a + 1):
        src = ctx + int(unpack[best, j])
        dst = ctx + j
        if src != dst:
            kv.k[:, dst] = kv.k[:, src]
            kv.v[:, dst] = kv.v[:, src]
    return ctx + 1 + a


# ----------------------------------------------------------------------------
# the whole step (Section 3.4) for one sequence
# ----------------------------------------------------------------------------
def spec_step(W, D, cfg, kv, ctx, g, h, beam_width, beam_length, planted=None,
              tree=True, dtype=F, run_drafter=True, sampling=None, seq=0, store=None):
    """One speculative decode step.  Returns a dict with every intermediate.

    planted: optional [BW, L] beams used in place of the drafter's (the drafter
    still runs when run_drafter is True, as in the timed planted-beam mode).
    """
    out = {}
    if run_drafter or planted is None:
        beams, scores = beam_search(D, W["tok_emb"], g, h, beam_width, beam_length, dtype, store=store)
        out["drafted_beams"], out["scores"] = beams, scores
    if planted is not None:
        beams = np.asarray(planted, dtype=np.int64)
    beam_aug = np.concatenate([np.full((beams.shape[0], 1), g, dtype=np.int64), beams], axis=1)
    packed = pack_beam(beam_aug, ctx) if tree else flat_beam(beam_aug, ctx)
    hidden, logits = llm_forward(W, cfg, packed["tokens"], packed["pos"], packed["mask"], kv, ctx, dtype, store=store)
    am = choose_rows(logits, packed["pos"], sampling, seq)
    a, best, emitted = accept_greedy(beams, packed["unpack"], am)
    node = int(packed["unpack"][best, a])
    new_ctx = compact_kv(kv, ctx, packed["unpack"], best, a)
    out.update(beams=beams, packed=packed, hidden=hidden, logits=logits, argmax=am,
               n_accept=a, best=best, emitted=emitted, ctx=new_ctx, g=emitted[-1],
               h=hidden[node].copy())
    return out


def generate_ar(W, cfg, prompt, n_tokens, max_ctx, dtype=F, sampling=None, seq=0, store=None):
    """Plain decoding (greedy, or sampled): the definition the speculative path must reproduce."""
    kv = KVCache(cfg["n_layers"], max_ctx, cfg["n_heads"], cfg["d_model"] // cfg["n_heads"], dtype)
    ctx, g, h = prefill(W, cfg, prompt, kv, dtype, sampling, seq, store)
    out = [g]
    while len(out) < n_tokens:
        nxt, h, _ = ar_step(W, cfg, kv, ctx, g, dtype, sampling, seq, store)
        ctx += 1
        g = nxt
        out.append(g)
    return out, kv, ctx


def generate_spec(W, D, cfg, prompt, n_steps, beam_width, beam_length, max_ctx,
                  planted_fn=None, tree=True, dtype=F, sampling=None, seq=0, store=None):
    """Speculative decoding for n_steps.  planted_fn(step, ctx, g) -> beams or None."""
    kv = KVCache(cfg["n_layers"], max_ctx, cfg["n_heads"], cfg["d_model"] // cfg["n_heads"], dtype)
    ctx, g, h = prefill(W, cfg, prompt, kv, dtype, sampling, seq, store)
    out = [g]
    accepted = []
    for step in range(n_steps):
        planted = planted_fn(step, len(out), g) if planted_fn is not None else None
        r = spec_step(W, D, cfg, kv, ctx, g, h, beam_width, beam_length, planted, tree, dtype,
                      run_drafter=planted is None, sampling=sampling, seq=seq, store=store)
        ctx, g, h = r["ctx"], r["g"], r["h"]
        out.extend(r["emitted"])
        accepted.append(r["n_accept"])
    return out, accepted, kv, ctx

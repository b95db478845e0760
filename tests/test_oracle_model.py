"""Pins for the oracle's drafter, beam search, LLM forward and the whole step
(Sections 3.1, 3.2, 3.4): closed forms, invariants, library cross-checks and the
lossless property."""
import itertools

import numpy as np
import torch

from helpers import first_mismatch, MICRO, micro_model
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth


# ------------------------------------------------------------------ elementary
def test_silu_logsoftmax_rmsnorm_against_torch():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(5, 37)) * 3
    tx = torch.from_numpy(x)
    assert np.allclose(ora.silu(x), torch.nn.functional.silu(tx).numpy(), atol=1e-12)
    for r in range(5):
        assert np.allclose(ora.log_softmax(x[r]), torch.log_softmax(tx[r], 0).numpy(), atol=1e-12)
        assert abs(np.exp(ora.log_softmax(x[r])).sum() - 1.0) < 1e-12
    g = rng.normal(size=37)
    ref = torch.nn.functional.rms_norm(tx, (37,), torch.from_numpy(g), eps=1e-6).numpy()
    assert np.allclose(ora.rmsnorm(x, g, 1e-6), ref, atol=1e-12)


def test_rope_properties():
    rng = np.random.default_rng(1)
    q = rng.normal(size=(1, 2, 16))
    k = rng.normal(size=(1, 2, 16))
    assert np.allclose(ora.rope(q, [0], 10000.0), q)                       # position 0 is the identity
    r = ora.rope(q, [13], 10000.0)
    assert np.allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(q, axis=-1))   # a rotation
    # relative-position property: <R(p)q, R(p')k> depends on p - p' only
    d1 = (ora.rope(q, [9], 1e4) * ora.rope(k, [4], 1e4)).sum(-1)
    d2 = (ora.rope(q, [25], 1e4) * ora.rope(k, [20], 1e4)).sum(-1)
    assert np.allclose(d1, d2)
    # pair (i, i + hd/2) rotates by pos * theta^(-2i/hd): check one pair explicitly
    x = np.zeros((1, 1, 8)); x[0, 0, 1] = 1.0
    y = ora.rope(x, [3], 100.0)
    ang = 3 * 100.0 ** (-2 * 1 / 8)
    assert np.allclose(y[0, 0, 1], np.cos(ang)) and np.allclose(y[0, 0, 5], np.sin(ang))
    assert np.count_nonzero(np.abs(y) > 1e-15) == 2


# ------------------------------------------------------------------ drafter
def test_rnn_cell_closed_forms():
    d = 8
    rng = np.random.default_rng(2)
    e = rng.normal(size=d); s = rng.normal(size=d)
    D = dict(rnn_u=np.zeros((d, d)), rnn_w=np.eye(d), rnn_b=np.zeros(d))
    assert np.allclose(ora.rnn_cell(D, s, e), e / (1 + np.exp(-e)))           # U=0, W=I: f(e)
    D = dict(rnn_u=np.eye(d), rnn_w=np.zeros((d, d)), rnn_b=np.full(d, 0.5))
    assert np.allclose(ora.rnn_cell(D, s, e), (s + .5) / (1 + np.exp(-(s + .5))))   # uses s, adds b
    U = rng.normal(size=(d, d)); Wm = rng.normal(size=(d, d))
    D = dict(rnn_u=U, rnn_w=Wm, rnn_b=np.zeros(d))
    z = np.array([sum(U[i, j] * s[j] for j in range(d)) + sum(Wm[i, j] * e[j] for j in range(d)) for i in range(d)])
    assert np.allclose(ora.rnn_cell(D, s, e), z / (1 + np.exp(-z)))           # U hits s, W hits e (not transposed)


def test_head_closed_forms():
    n, V = 6, 5
    rng = np.random.default_rng(3)
    x = rng.normal(size=n)
    O = rng.normal(size=(V, n))
    zero = dict(head_w=[np.zeros((n, n))] * 2, head_b=[np.zeros(n)] * 2, draft_out=O)
    assert np.allclose(ora.draft_head(zero, x), O @ x)                        # A=0,c=0: SiLU(0)=0, skip path only
    c = rng.normal(size=n)
    one = dict(head_w=[np.zeros((n, n))], head_b=[c], draft_out=np.eye(n))
    assert np.allclose(ora.draft_head(one, x), x + c / (1 + np.exp(-c)))      # skip + SiLU(bias)
    A = rng.normal(size=(n, n))
    lin = dict(head_w=[A], head_b=[np.zeros(n)], draft_out=np.eye(n))
    z = A @ x
    assert np.allclose(ora.draft_head(lin, x), x + z / (1 + np.exp(-z)))


def test_beam_width_one_is_greedy_drafting():
    cfg, W, D, _ = micro_model()
    rng = np.random.default_rng(4)
    h = rng.normal(size=cfg["d_model"])
    g = 5
    beams, scores = ora.beam_search(D, W["tok_emb"], g, h, 1, 4)
    E = W["tok_emb"].astype(np.float64)
    s, seq, tot = E[g], [], 0.0
    for t in range(4):
        if t > 0:
            s = ora.rnn_cell(D, s, E[seq[-1]])
        lp = ora.log_softmax(ora.draft_head(D, np.concatenate([s, h])))
        seq.append(int(np.argmax(lp))); tot += lp.max()
    assert beams[0].tolist() == seq and abs(scores[0] - tot) < 1e-10


def test_beam_scores_and_order():
    cfg, W, D, _ = micro_model()
    rng = np.random.default_rng(5)
    h = rng.normal(size=cfg["d_model"])
    beams, scores = ora.beam_search(D, W["tok_emb"], 9, h, 6, 4)
    assert (np.diff(scores) <= 0).all()
    assert len({tuple(b) for b in beams}) == 6
    for b, s in zip(beams, scores):
        assert abs(ora.sequence_logprob(D, W["tok_emb"], 9, h, b) - s) < 1e-9


def test_beam_search_exhaustive_tiny_vocab():
    cfg = dict(MICRO, vocab=8, d_model=16, n_heads=2, d_ffn=24, d_rnn=16)
    cfg, W, D, _ = micro_model(std=0.6, cfg=cfg)
    h = np.random.default_rng(6).normal(size=16)
    # L=2 with BW = V keeps every first token alive, so the beam is the exact top-8 of all 64 sequences
    beams, scores = ora.beam_search(D, W["tok_emb"], 3, h, 8, 2)
    allseq = list(itertools.product(range(8), repeat=2))
    lps = np.array([ora.sequence_logprob(D, W["tok_emb"], 3, h, s) for s in allseq])
    order = np.argsort(-lps, kind="stable")[:8]
    assert [allseq[i] for i in order] == [tuple(b) for b in beams]
    assert np.allclose(lps[order], scores)
    assert abs(np.exp(lps).sum() - 1.0) < 1e-9                               # a distribution over sequences


# ------------------------------------------------------------------ LLM forward
def _torch_llama(W, cfg, tokens):
    """Causal forward written with torch library routines (rms_norm, SDPA with a boolean mask)."""
    Fn = torch.nn.functional
    d, H = cfg["d_model"], cfg["n_heads"]; hd = d // H
    n = len(tokens)
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    x = t(W["tok_emb"])[torch.tensor(tokens)]
    pos = torch.arange(n, dtype=torch.float64)
    inv = cfg["rope_theta"] ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd)
    ang = pos[:, None] * inv[None, :]
    cos = torch.cat([ang.cos(), ang.cos()], -1)[None]; sin = torch.cat([ang.sin(), ang.sin()], -1)[None]
    rot = lambda v: torch.cat([-v[..., hd // 2:], v[..., :hd // 2]], -1)
    causal = torch.tril(torch.ones(n, n, dtype=torch.bool))
    for l in range(cfg["n_layers"]):
        a = Fn.rms_norm(x, (d,), t(W["attn_norm"][l]), eps=cfg["rms_eps"])
        qkv = a @ t(W["wqkv"][l]).T
        q, k, v = [z.reshape(n, H, hd).transpose(0, 1) for z in qkv.split(d, dim=1)]
        q = q * cos + rot(q) * sin; k = k * cos + rot(k) * sin
        o = Fn.scaled_dot_product_attention(q, k, v, attn_mask=causal).transpose(0, 1).reshape(n, d)
        x = x + o @ t(W["wo"][l]).T
        f = Fn.rms_norm(x, (d,), t(W["ffn_norm"][l]), eps=cfg["rms_eps"])
        gu = f @ t(W["w_gate_up"][l]).T
        x = x + (Fn.silu(gu[:, :cfg["d_ffn"]]) * gu[:, cfg["d_ffn"]:]) @ t(W["w_down"][l]).T
    hid = Fn.rms_norm(x, (d,), t(W["final_norm"]), eps=cfg["rms_eps"])
    return hid.numpy(), (hid @ t(W["lm_head"]).T).numpy()


def test_llm_forward_against_torch_library_routines():
    cfg, W, D, _ = micro_model()
    toks = np.random.default_rng(7).integers(0, cfg["vocab"], size=11)
    kv = ora.KVCache(cfg["n_layers"], 32, cfg["n_heads"], 16)
    hid, logits = ora.llm_forward(W, cfg, toks, np.arange(11), np.tril(np.ones((11, 11), bool)), kv, 0)
    rh, rl = _torch_llama(W, cfg, toks.tolist())
    assert np.allclose(hid, rh, atol=1e-9) and np.allclose(logits, rl, atol=1e-9)


def test_incremental_equals_full_causal():
    """A forward over [cache | new rows] equals the tail of one causal forward (N=1: an AR step)."""
    cfg, W, D, _ = micro_model()
    toks = np.random.default_rng(8).integers(0, cfg["vocab"], size=10)
    kv_full = ora.KVCache(cfg["n_layers"], 32, cfg["n_heads"], 16)
    _, full = ora.llm_forward(W, cfg, toks, np.arange(10), np.tril(np.ones((10, 10), bool)), kv_full, 0)
    kv = ora.KVCache(cfg["n_layers"], 32, cfg["n_heads"], 16)
    ora.llm_forward(W, cfg, toks[:7], np.arange(7), np.tril(np.ones((7, 7), bool)), kv, 0)
    _, l7 = ora.llm_forward(W, cfg, toks[7:8], [7], np.ones((1, 1), bool), kv, 7)
    assert np.allclose(l7[0], full[7], atol=1e-10)
    _, tail = ora.llm_forward(W, cfg, toks[8:], [8, 9], np.tril(np.ones((2, 2), bool)), kv, 8)
    assert np.allclose(tail, full[8:], atol=1e-10)
    assert np.allclose(kv.k[:, :10], kv_full.k[:, :10], atol=1e-10)


def test_packed_tree_equals_per_beam_causal():
    cfg, W, D, _ = micro_model()
    rng = np.random.default_rng(9)
    prompt = rng.integers(0, cfg["vocab"], size=9)
    kv = ora.KVCache(cfg["n_layers"], 64, cfg["n_heads"], 16)
    ctx, g, h = ora.prefill(W, cfg, prompt, kv)
    beams = rng.integers(0, 3, size=(5, 4))                 # a small alphabet forces shared prefixes
    aug = np.concatenate([np.full((5, 1), g), beams], axis=1)
    p = ora.pack_beam(aug, ctx)
    assert p["n"] < 1 + 5 * 4
    _, logits = ora.llm_forward(W, cfg, p["tokens"], p["pos"], p["mask"], kv, ctx)
    for i in range(5):
        kvi = ora.KVCache(cfg["n_layers"], 64, cfg["n_heads"], 16)
        kvi.k[:, :ctx] = kv.k[:, :ctx]; kvi.v[:, :ctx] = kv.v[:, :ctx]
        _, li = ora.llm_forward(W, cfg, aug[i], ctx + np.arange(5), np.tril(np.ones((5, 5), bool)), kvi, ctx)
        assert np.allclose(logits[p["unpack"][i]], li, atol=1e-10)
    # and the no-tree-attention arm gives the same per-node logits
    pf = ora.flat_beam(aug, ctx)
    _, lf = ora.llm_forward(W, cfg, pf["tokens"], pf["pos"], pf["mask"], kv, ctx)
    for i in range(5):
        assert np.allclose(lf[pf["unpack"][i]], logits[p["unpack"][i]], atol=1e-10)


# ------------------------------------------------------------------ whole step
def _planted_fn(ar_tokens, cfg, rng, p, rho):
    def fn(step, n_out, g):
        return synth.plant_beams(ar_tokens[n_out:n_out + cfg["beam_length"]], cfg["beam_width"],
                                 cfg["beam_length"], cfg["vocab"], rng, p=p, rho=rho)
    return fn


def test_lossless_drafted_and_planted_and_cache():
    cfg, W, D, _ = micro_model()
    prompt = synth.make_prompts(cfg, 1)[0]
    n_steps = 8
    ar, kv_ar, ctx_ar = ora.generate_ar(W, cfg, prompt, 1 + n_steps * (cfg["beam_length"] + 1), cfg["max_ctx"])
    # drafter's own beams (random-init drafter: mostly a = 0)
    out, acc, kv, ctx = ora.generate_spec(W, D, cfg, prompt, n_steps, 4, 4, cfg["max_ctx"])
    assert out == ar[:len(out)]
    assert len(out) == 1 + sum(a + 1 for a in acc)
    # planted beams: acceptance is exercised, output still identical, accepted length = closed form
    rng = np.random.default_rng(10)
    out, acc, kv, ctx = ora.generate_spec(W, D, cfg, prompt, n_steps, 4, 4, cfg["max_ctx"],
                                          planted_fn=_planted_fn(ar, cfg, rng, 0.3, 0.5))
    assert out == ar[:len(out)]
    assert max(acc) >= 2 and min(acc) < 4
    rng = np.random.default_rng(10)
    pos = 1
    for a in acc:
        b = synth.plant_beams(ar[pos:pos + 4], 4, 4, cfg["vocab"], rng, p=0.3, rho=0.5)
        assert a == first_mismatch(b, ar[pos:pos + 4]).max()
        pos += a + 1
    # compaction: the cache after speculative decoding equals the AR cache over the same tokens
    n = min(ctx, ctx_ar)
    assert np.allclose(kv.k[:, :n], kv_ar.k[:, :n], atol=1e-9)
    assert np.allclose(kv.v[:, :n], kv_ar.v[:, :n], atol=1e-9)
    # the no-tree-attention arm is lossless too
    out2, _, _, _ = ora.generate_spec(W, D, cfg, prompt, 3, 4, 4, cfg["max_ctx"], tree=False)
    assert out2 == ar[:len(out2)]


def test_lossless_tiny_config_fp64():
    cfg = dict(synth.CONFIGS["tiny"])
    w = synth.make_weights(cfg, "cpu")
    W, D = synth.weights_to_numpy(w, cfg)
    prompt = synth.make_prompts(cfg, 1)[0]
    steps = 6
    ar, _, _ = ora.generate_ar(W, cfg, prompt, 1 + steps * 5, cfg["max_ctx"])
    rng = np.random.default_rng(11)
    out, acc, _, _ = ora.generate_spec(W, D, cfg, prompt, steps, 4, 4, cfg["max_ctx"],
                                       planted_fn=_planted_fn(ar, cfg, rng, 0.3, 0.0))
    assert out == ar[:len(out)] and sum(acc) > 0

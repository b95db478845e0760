"""Seeded synthetic inputs: model shapes, random-init weights, prompts, planted beams.

This module serves both the CUDA path and the test oracle and therefore holds none
of the method's arithmetic: it only draws random numbers and arranges them.  The
shapes stand in for the Vicuna 7B/13B/33B models and the prompts for the MT-Bench /
AlpacaEval prompts the paper measures on (Section 4); neither is available offline.
"""
from __future__ import annotations

import numpy as np
import torch

WEIGHT_SEED = 20240309


def _cfg(n_layers, d_model, n_heads, d_ffn, vocab, dtype, max_batch, max_ctx, beam_width,
         beam_length, prompt_len, steps, **extra):
    c = dict(n_layers=n_layers, d_model=d_model, n_heads=n_heads, d_ffn=d_ffn, vocab=vocab,
             rms_eps=1e-6, rope_theta=10000.0, d_rnn=d_model, n_head_layers=2, dtype=dtype,
             max_batch=max_batch, max_ctx=max_ctx, beam_width=beam_width, beam_length=beam_length,
             prompt_len=prompt_len, steps=steps)
    c.update(extra)
    return c


# The five workloads.  prompt_len is an int or an inclusive (lo, hi) range for ragged batches.
CONFIGS = {
    "tiny": _cfg(2, 256, 4, 688, 1024, "fp32", 1, 64 + 32 * 5 + 24, 4, 4, 64, 32, seed=1),
    "7b": _cfg(32, 4096, 32, 11008, 32000, "bf16", 1, 512 + 256 * 6 + 48, 8, 5, 512, 256, seed=2),
    "13b": _cfg(40, 5120, 40, 13824, 32000, "bf16", 1, 1024 + 128 * 6 + 328, 64, 5, 1024, 128, seed=3,
                plant_p=0.3, plant_rho=0.5),
    "7b_bs16": _cfg(32, 4096, 32, 11008, 32000, "bf16", 16, 2048 + 128 * 6 + 88, 16, 5, (256, 2048), 128, seed=4),
    "33b": _cfg(60, 6656, 52, 17920, 32000, "bf16", 4, 4096 + 64 * 6 + 168, 32, 5, 4096, 64, seed=5),
}


def with_layers(cfg, n_layers):
    """A depth-reduced copy: full per-layer shapes, fewer layers."""
    c = dict(cfg)
    c["n_layers"] = n_layers
    return c


def weight_shapes(cfg):
    """Name -> (shape, kind) for every tensor of the target LLM and the drafter."""
    d, Fd, V, dr = cfg["d_model"], cfg["d_ffn"], cfg["vocab"], cfg["d_rnn"]
    dh = dr + d
    s = {"tok_emb": ((V, d), "w"), "final_norm": ((d,), "g"), "lm_head": ((V, d), "w")}
    for l in range(cfg["n_layers"]):
        s[f"attn_norm.{l}"] = ((d,), "g")
        s[f"wqkv.{l}"] = ((3 * d, d), "w")
        s[f"wo.{l}"] = ((d, d), "w")
        s[f"ffn_norm.{l}"] = ((d,), "g")
        s[f"w_gate_up.{l}"] = ((2 * Fd, d), "w")
        s[f"w_down.{l}"] = ((d, Fd), "w")
    s["rnn_u"] = ((dr, dr), "w")
    s["rnn_w"] = ((dr, d), "w")
    s["rnn_b"] = ((dr,), "w")
    for l in range(cfg["n_head_layers"]):
        s[f"head_w.{l}"] = ((dh, dh), "w")
        s[f"head_b.{l}"] = ((dh,), "w")
    s["draft_out"] = ((V, dh), "w")
    return s


def make_weights(cfg, device="cpu", seed=WEIGHT_SEED, std=0.02, gain_jitter=0.0):
    """Every matrix and bias ~ N(0, std); norm gains 1 (+ optional jitter so tests see a
    non-trivial gain).  Returned in the config's storage dtype on `device`."""
    tdt = torch.float32 if cfg["dtype"] == "fp32" else torch.bfloat16
    out = {}
    for idx, (name, (shape, kind)) in enumerate(weight_shapes(cfg).items()):
        gen = torch.Generator(device=device)
        gen.manual_seed(seed + idx)
        if kind == "g":
            t = torch.ones(shape, device=device, dtype=torch.float32)
            if gain_jitter:
                t = t + gain_jitter * torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        else:
            t = torch.empty(shape, device=device, dtype=torch.float32).normal_(0.0, std, generator=gen)
        out[name] = t.to(tdt)
    return out


def weights_to_numpy(weights, cfg):
    """Host float32 copies of the stored values, grouped the way a reader of the paper
    would name them: (LLM dict, drafter dict)."""
    def np32(t):
        return t.detach().to("cpu", torch.float32).numpy()
    L = cfg["n_layers"]
    W = {"tok_emb": np32(weights["tok_emb"]), "final_norm": np32(weights["final_norm"]),
         "lm_head": np32(weights["lm_head"])}
    for k in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down"):
        W[k] = [np32(weights[f"{k}.{l}"]) for l in range(L)]
    D = {"rnn_u": np32(weights["rnn_u"]), "rnn_w": np32(weights["rnn_w"]), "rnn_b": np32(weights["rnn_b"]),
         "head_w": [np32(weights[f"head_w.{l}"]) for l in range(cfg["n_head_layers"])],
         "head_b": [np32(weights[f"head_b.{l}"]) for l in range(cfg["n_head_layers"])],
         "draft_out": np32(weights["draft_out"])}
    return W, D


def make_prompts(cfg, batch=None, seed=None):
    """Tokens uniform over the vocabulary; ragged lengths when prompt_len is a range."""
    rng = np.random.Generator(np.random.PCG64(1000 + (cfg.get("seed", 0) if seed is None else seed)))
    batch = cfg["max_batch"] if batch is None else batch
    pl = cfg["prompt_len"]
    prompts = []
    for _ in range(batch):
        n = int(pl) if isinstance(pl, int) else int(rng.integers(pl[0], pl[1] + 1))
        prompts.append(rng.integers(0, cfg["vocab"], size=n, dtype=np.int64))
    return prompts


def plant_beams(continuation, beam_width, beam_length, vocab, rng, p=0.3, rho=0.0):
    """Planted beams: every candidate is the given continuation (the target's own greedy
    tokens) with each position independently replaced, with probability p, by a
    different token; with probability rho a candidate i > 0 first copies a prefix of
    random length in [1, L-1] from a uniformly chosen earlier candidate."""
    cont = np.asarray(continuation[:beam_length], dtype=np.int64)
    assert cont.shape[0] == beam_length
    beams = np.zeros((beam_width, beam_length), dtype=np.int64)
    for i in range(beam_width):
        row = cont.copy()
        repl = rng.random(beam_length) < p
        r = rng.integers(0, vocab - 1, size=beam_length)
        row[repl] = (cont[repl] + 1 + r[repl]) % vocab
        if i > 0 and rho > 0.0 and rng.random() < rho and beam_length > 1:
            src = int(rng.integers(0, i))
            ell = int(rng.integers(1, beam_length))
            row[:ell] = beams[src, :ell]
        beams[i] = row
    return beams


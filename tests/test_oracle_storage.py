"""Pins of the oracle's store="bf16" mode (CPU only).

The bf16 configurations keep some intermediates in bfloat16 (every projection input, Q, K, V, the softmax weights
that multiply V).  The oracle can round exactly those arrays; these tests tie that mode to things fixed outside it:
the bit-level definition of round-to-nearest-even, a library cast, the properties the unrounded oracle is pinned by
(which rounding element by element must preserve), and the size of the storage error and its growth with depth --
the figure the full-depth GPU parity tests rely on.
"""
import numpy as np
import pytest
import torch

from helpers import micro_model
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth


# ------------------------------------------------------------------ the rounding itself
def test_round_bf16_known_values():
    # bfloat16 keeps 8 significant bits: the spacing in [1, 2) is 2^-7
    e = 2.0 ** -7
    cases = [
        (1.0, 1.0),
        (1.0 + e, 1.0 + e),
        (1.0 + e / 2, 1.0),                    # a tie goes to the even significand
        (1.0 + 3 * e / 2, 1.0 + 2 * e),        # ... here upwards
        (1.0 + e / 2 + 2.0 ** -20, 1.0 + e),   # just above a tie
        (1.0 + e / 2 - 2.0 ** -20, 1.0),       # just below
        (-1.0 - 3 * e / 2, -1.0 - 2 * e),      # sign symmetric
        (0.0, 0.0),
        (2.0 ** 127 * (1 + e / 2), 2.0 ** 127),   # the same tie at the top of the exponent range
        (np.inf, np.inf),
        (2.0 ** -130, 2.0 ** -130),            # a float32 subnormal that bfloat16 represents exactly
    ]
    for x, want in cases:
        got = float(ora.round_bf16(np.array([x], dtype=np.float64))[0])
        assert got == want, (x, got, want)


def test_round_bf16_against_the_bit_definition_and_a_library_cast():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000), rng.standard_normal(2000) * 1e-30, rng.standard_normal(2000) * 1e20,
                        np.ldexp(rng.integers(128, 256, size=2000) + 0.5, rng.integers(-40, 40, size=2000))]).astype(np.float32)
    got = ora.round_bf16(x)
    assert got.dtype == np.float32
    # (a) the definition: the nearest value with 16 zero low bits; on a tie the one whose bit 16 is zero
    u = x.view(np.uint32).astype(np.uint64)
    down = u & np.uint64(0xFFFF0000)
    up = down + np.uint64(0x10000)
    rem = u & np.uint64(0xFFFF)
    pick_up = (rem > 0x8000) | ((rem == 0x8000) & ((down >> np.uint64(16)) & np.uint64(1)).astype(bool))
    want = np.where(pick_up, up, down).astype(np.uint32).view(np.float32)
    assert (got.view(np.uint32) == want.view(np.uint32)).all()
    # (b) torch's cast
    lib = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert (got.view(np.uint32) == lib.view(np.uint32)).all()
    # idempotent, and the identity on values that already are bfloat16
    assert (ora.round_bf16(got) == got).all()
    # from float64 the value passes through float32 first, as the stored intermediates do
    x64 = rng.standard_normal(1000)
    assert (ora.round_bf16(x64) == ora.round_bf16(x64.astype(np.float32)).astype(np.float64)).all()
    assert ora.round_bf16(x64).dtype == np.float64


# ------------------------------------------------------------------ the rounded forward keeps the oracle's own pins
def test_rounded_mode_keeps_packed_equals_per_beam_and_lossless():
    cfg, W, D, _ = micro_model()
    prompt = np.random.default_rng(3).integers(0, cfg["vocab"], size=cfg["prompt_len"])
    hd = cfg["d_model"] // cfg["n_heads"]
    ar, _, _ = ora.generate_ar(W, cfg, prompt, 30, cfg["max_ctx"], store="bf16")
    ar_plain, _, _ = ora.generate_ar(W, cfg, prompt, 30, cfg["max_ctx"])
    # rounding is element-wise, so a packed node and the same node in a per-candidate run see identical numbers
    kv = ora.KVCache(cfg["n_layers"], cfg["max_ctx"], cfg["n_heads"], hd)
    ctx, g, h = ora.prefill(W, cfg, prompt, kv, store="bf16")
    assert g == ar[0]
    beams = synth.plant_beams(ar[1:5], 4, 4, cfg["vocab"], np.random.default_rng(4), p=0.3, rho=0.4)
    aug = np.concatenate([np.full((4, 1), g), beams], axis=1)
    p = ora.pack_beam(aug, ctx)
    kv1 = ora.KVCache(cfg["n_layers"], cfg["max_ctx"], cfg["n_heads"], hd)
    kv1.k[:], kv1.v[:] = kv.k, kv.v
    _, packed_logits = ora.llm_forward(W, cfg, p["tokens"], p["pos"], p["mask"], kv1, ctx, store="bf16")
    for i in range(4):
        kv2 = ora.KVCache(cfg["n_layers"], cfg["max_ctx"], cfg["n_heads"], hd)
        kv2.k[:], kv2.v[:] = kv.k, kv.v
        _, lg = ora.llm_forward(W, cfg, aug[i], ctx + np.arange(5), np.tril(np.ones((5, 5), bool)), kv2, ctx, store="bf16")
        assert (lg == packed_logits[p["unpack"][i]]).all()
    # and the speculative stream still is the plain stream of the same (rounded) model, token for token
    rng = np.random.default_rng(5)
    out, acc, _, _ = ora.generate_spec(
        W, D, cfg, prompt, 5, 4, 4, cfg["max_ctx"], store="bf16",
        planted_fn=lambda step, n_out, g_: synth.plant_beams(ar[n_out:n_out + 4], 4, 4, cfg["vocab"], rng, p=0.3))
    assert out == ar[:len(out)] and max(acc) >= 2
    # the rounded model is a different function: its logits differ from the plain ones, by about a bf16 step
    kv3 = ora.KVCache(cfg["n_layers"], cfg["max_ctx"], cfg["n_heads"], hd)
    ora.prefill(W, cfg, prompt, kv3)
    kv4 = ora.KVCache(cfg["n_layers"], cfg["max_ctx"], cfg["n_heads"], hd)
    ora.prefill(W, cfg, prompt, kv4, store="bf16")
    rel = np.abs(kv3.k[:, :ctx] - kv4.k[:, :ctx]).max() / np.abs(kv3.k[:, :ctx]).max()
    assert 1e-4 < rel < 2e-2
    # every stored K/V entry is a bfloat16 value
    assert (ora.round_bf16(kv4.k[:, :ctx]) == kv4.k[:, :ctx]).all() and (ora.round_bf16(kv4.v[:, :ctx]) == kv4.v[:, :ctx]).all()
    del ar_plain


def test_rounded_drafter_scores_are_sequence_logprobs_of_the_rounded_drafter():
    cfg, W, D, _ = micro_model()
    rng = np.random.default_rng(6)
    h = rng.standard_normal(cfg["d_model"])
    beams, scores = ora.beam_search(D, W["tok_emb"], 5, h, 4, 4, store="bf16")
    for b, s in zip(beams, scores):
        assert abs(ora.sequence_logprob(D, W["tok_emb"], 5, h, b, store="bf16") - s) < 1e-9
    plain = [ora.sequence_logprob(D, W["tok_emb"], 5, h, b) for b in beams]
    d = np.abs(np.array(plain) - scores)
    assert 1e-6 < d.max() < 0.2          # a different function, by a rounding-sized amount
    # beam width 1 is the greedy chain of the rounded drafter
    b1, s1 = ora.beam_search(D, W["tok_emb"], 5, h, 1, 4, store="bf16")
    E = W["tok_emb"].astype(np.float64)
    s, toks = E[5], []
    for t in range(4):
        if t:
            s = ora.rnn_cell(D, s, E[toks[-1]], store="bf16")
        toks.append(int(np.argmax(ora.draft_head(D, np.concatenate([s, h]), store="bf16"))))
    assert b1[0].tolist() == toks


# ------------------------------------------------------------------ what the storage costs, and how it grows with depth
def test_storage_error_grows_as_sqrt_depth_at_the_7b_layer_shape():
    """Random-init layers of the 7B shape (d 4096, 32 heads, FFN 11008; vocabulary cut to 4096 to bound the test's
    memory): relative L2 distance between the logits of the rounded and the unrounded oracle after 1, 2, 4 and 8
    layers.  The rounding noise of different layers is independent and the layers neither damp nor amplify it much,
    so it grows like sqrt(depth): 0.7e-2 after one layer, 1.6e-2 after eight, which extrapolates to 3e-2 for the
    average row (more for the worst row and the worst element) at the 32 layers of the 7B workload and beyond it at
    40 and 60 layers.  This is a property of the precision, measured without any kernel: the full-depth GPU parity
    cases are therefore held to the stated 3e-2 against the ROUNDED oracle, and their distance to the unrounded one is
    reported, not bounded by 3e-2."""
    cfg = dict(synth.CONFIGS["7b"], n_layers=8, vocab=4096, n_head_layers=0, max_ctx=32)
    W, _ = synth.weights_to_numpy(synth.make_weights(cfg, "cpu"), cfg)
    prompt = np.random.default_rng(0).integers(0, cfg["vocab"], size=24)
    P = len(prompt)
    mask = np.tril(np.ones((P, P), bool))
    err = {}
    for depth in (1, 2, 4, 8):
        c = dict(cfg, n_layers=depth)
        lg = []
        for store in (None, "bf16"):
            kv = ora.KVCache(depth, 32, cfg["n_heads"], 128, np.float32)
            lg.append(ora.llm_forward(W, c, prompt, np.arange(P), mask, kv, 0, np.float32, store=store)[1])
        err[depth] = float(np.mean(np.linalg.norm(lg[0] - lg[1], axis=1) / np.linalg.norm(lg[0], axis=1)))
    assert 0.4e-2 < err[1] < 1.0e-2
    for depth in (2, 4, 8):
        # within 25 % of err[1] * sqrt(depth); linear growth (x depth) or none would both fail
        assert 0.75 < err[depth] / (err[1] * np.sqrt(depth)) < 1.25, err
    # extrapolated to the workloads' depths the storage alone exceeds the 3e-2 that holds for shallow copies
    assert err[8] * np.sqrt(32 / 8) > 2.5e-2

    # Two correct implementations of the SAME rounded arithmetic drift apart: perturb every array by a relative 1e-6
    # before it is rounded (what a different summation order does to an fp32 sum) and the logits after eight layers
    # differ from the unperturbed rounded run by more than half the storage noise itself, while both stay equally far
    # from the unrounded oracle.  A tight bound against the rounded oracle is therefore not a property any kernel can
    # have; the GPU parity cases bound the distance to BOTH oracle modes by the distance between them.
    def mean_l2(a, b):
        return float(np.mean(np.linalg.norm(a - b, axis=1) / np.linalg.norm(b, axis=1)))
    rng = np.random.default_rng(1)
    plain_st = ora._st

    def jittered_st(a, store):
        if store is None:
            return a
        return ora.round_bf16(a * (1 + 1e-6 * rng.standard_normal(a.shape).astype(a.dtype)))
    c = dict(cfg, n_layers=8)
    runs = {}
    for name, st, store in (("U", plain_st, None), ("R", plain_st, "bf16"), ("R2", jittered_st, "bf16")):
        ora._st = st
        try:
            kv = ora.KVCache(8, 32, cfg["n_heads"], 128, np.float32)
            runs[name] = ora.llm_forward(W, c, prompt, np.arange(P), mask, kv, 0, np.float32, store=store)[1]
        finally:
            ora._st = plain_st
    noise = mean_l2(runs["R"], runs["U"])
    assert 0.5 * noise < mean_l2(runs["R2"], runs["R"]) < 1.1 * noise
    assert abs(mean_l2(runs["R2"], runs["U"]) - noise) < 0.05 * noise

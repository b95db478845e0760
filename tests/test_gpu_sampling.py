"""Parity of the CUDA path's token choice at temperature > 0 with the oracle (Section 3.4: acceptance by rejection
sampling, read for deterministic proposals as the LLM's own draw at every tree node).

The draw is an argmax of (logit / T + Gumbel noise), i.e. a float decides an integer: tokens are compared where the
oracle's top-2 gap of those perturbed scores exceeds the bound that the logits' tolerance allows.  Everything that
follows from the tokens (accepted length, winner, emitted tokens, state) is compared bit-exactly.
"""
import numpy as np
import pytest
import torch

from helpers import Rig, dev, top2_gap
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu

GAP = 0.05
TOL_FP32 = 2e-3
SMP = dict(temperature=0.8, seed=(5 << 32) + 17)          # both halves of the seed in use

BF16 = dict(synth.CONFIGS["tiny"], dtype="bf16", d_model=512, n_heads=4, d_ffn=1376, vocab=1000, d_rnn=512,
            max_ctx=400, beam_width=8, beam_length=5, prompt_len=96)


def oracle_draws(logits, pos, smp, seq):
    """(tokens, top-2 gap of the perturbed scores) per row; row r chooses the token at position pos[r] + 1."""
    toks, gaps = [], []
    for r in range(logits.shape[0]):
        t, z = ora.choose_token(logits[r], smp, seq, int(pos[r]) + 1, want_scores=True)
        toks.append(t)
        gaps.append(top2_gap(z))
    return np.array(toks), np.array(gaps)


@pytest.mark.parametrize("cfg,odt", [(None, np.float64), (BF16, np.float64)])
def test_draws_of_a_verification_pass(cfg, odt):
    B = 3
    r = Rig(cfg=cfg, max_batch=B, oracle_dtype=odt) if cfg is not None else Rig(max_batch=B)
    c = r.cfg
    BW, L, T = c["beam_width"], c["beam_length"], SMP["temperature"]
    rng = np.random.default_rng(21)
    prompts = [rng.integers(0, c["vocab"], size=n) for n in (40, 23, 64)]
    r.eng.set_sampling(T, SMP["seed"])
    r.eng.prefill(prompts)
    ctx_g, root_g, _ = r.eng.get_state()
    beams = rng.integers(0, 3, size=(B, BW, L))
    pk = r.eng.pack(dev(beams))
    toks, hidden, logits = r.eng.verify(pk, want_logits=True)
    r.eng.poll()
    compared_own = compared_ref = 0
    for b in range(B):
        kv = r.new_kv()
        ctx, g, h = ora.prefill(r.W, c, prompts[b], kv, r.odt, SMP, seq=b)
        assert int(ctx_g[b]) == ctx
        g_gpu = int(root_g[b])
        aug = np.concatenate([np.full((BW, 1), g_gpu), beams[b]], axis=1)
        p = ora.pack_beam(aug, ctx)
        n = p["n"]
        got = toks[b, :n].cpu().numpy()
        assert (toks[b, n:] == -1).all()
        # (1) the sampler alone: the oracle's rule applied to the GPU's own logits
        own = logits[b, :n].cpu().numpy().astype(np.float64)
        t_own, gap_own = oracle_draws(own, p["pos"], SMP, b)
        sure = gap_own > 1e-3
        assert (got[sure] == t_own[sure]).all()
        compared_own += int(sure.sum())
        # (2) end to end against the oracle's logits (same root on both sides)
        _, rl = ora.llm_forward(r.W, c, p["tokens"], p["pos"], p["mask"], kv, ctx, r.odt)
        t_ref, gap_ref = oracle_draws(rl, p["pos"], SMP, b)
        bound = (TOL_FP32 if c["dtype"] == "fp32" else 3e-2 * np.abs(rl).max(axis=-1)) / T
        sure = gap_ref > np.maximum(GAP, 2 * bound)
        assert (got[sure] == t_ref[sure]).all()
        compared_ref += int(sure.sum())
        # rows that choose the token of the same position share their noise: equal logits rows would agree; at least
        # the draws are not the greedy tokens everywhere
    assert compared_own >= 0.9 * sum(int(pk.n[b]) for b in range(B))
    assert compared_ref >= (12 if c["dtype"] == "fp32" else 6)
    greedy = logits.cpu().numpy().argmax(-1)
    drawn = toks.cpu().numpy()
    valid = drawn >= 0
    assert (drawn[valid] != greedy[valid]).any()
    r.eng.close()


def test_draws_at_7b_shapes_on_the_gpus_own_logits():
    """Vocabulary 32000, two sequences, tensor-core LM head with partial sums folded by the sampling kernel: the
    oracle's rule applied to the logits the GPU returns must give the GPU's tokens."""
    B = 2
    r = Rig(cfg=synth.with_layers(dict(synth.CONFIGS["7b"], max_ctx=256, max_batch=B), 2), oracle_dtype=np.float32)
    c = r.cfg
    BW, L = c["beam_width"], c["beam_length"]
    rng = np.random.default_rng(22)
    r.eng.set_sampling(1.3, 77)
    r.eng.prefill([rng.integers(0, c["vocab"], size=n) for n in (50, 31)])
    ctx_g, root_g, _ = r.eng.get_state()
    beams = rng.integers(0, 3, size=(B, BW, L))
    pk = r.eng.pack(dev(beams))
    toks, _, logits = r.eng.verify(pk, want_logits=True)
    r.eng.poll()
    smp = dict(temperature=1.3, seed=77)
    for b in range(B):
        n = int(pk.n[b])
        pos = pk.pos[b, :n].cpu().numpy()
        assert pos[0] == int(ctx_g[b])
        t_own, gap_own = oracle_draws(logits[b, :n].cpu().numpy().astype(np.float64), pos, smp, b)
        sure = gap_own > 1e-3
        assert sure.sum() >= n - 2
        assert (toks[b, :n].cpu().numpy()[sure] == t_own[sure]).all()
    r.eng.close()


def test_root_after_the_prompt_is_a_draw():
    r = Rig()
    prompt = synth.make_prompts(r.cfg, 1)[0]
    roots = set()
    for seed in range(6):
        smp = dict(temperature=1.0, seed=seed)
        r.eng.set_sampling(1.0, seed)
        r.eng.prefill([prompt])
        _, root, h = r.eng.get_state()
        r.eng.poll()
        kv = r.new_kv()
        P, g, hh = ora.prefill(r.W, r.cfg, prompt, kv, sampling=smp)
        lg = hh @ r.W["lm_head"].T
        _, z = ora.choose_token(lg, smp, 0, P, want_scores=True)
        if top2_gap(z) > GAP:
            assert int(root[0]) == g
        roots.add(int(root[0]))
    assert len(roots) > 1
    r.eng.close()


def test_steps_teacher_forced_with_sampling():
    r = Rig()
    cfg = r.cfg
    BW, L = cfg["beam_width"], cfg["beam_length"]
    prompt = synth.make_prompts(cfg, 1)[0]
    n_steps = 10
    r.eng.set_sampling(SMP["temperature"], SMP["seed"])
    r.eng.prefill([prompt])
    kv = r.new_kv()
    ctx, g, h = ora.prefill(r.W, cfg, prompt, kv, sampling=SMP)
    plain, _, _ = ora.generate_ar(r.W, cfg, prompt, 2 + n_steps * (L + 1), cfg["max_ctx"], sampling=SMP)
    assert plain[0] == g
    rng = np.random.default_rng(31)
    out = r.binding.AcceptOut(1, L, "cuda:0")
    emitted, accepted, checked = [g], [], 0
    for step in range(n_steps):
        planted = synth.plant_beams(plain[len(emitted):len(emitted) + L], BW, L, cfg["vocab"], rng, p=0.3, rho=0.3)
        ref = ora.spec_step(r.W, r.D, cfg, kv, ctx, g, h, BW, L, planted=planted, run_drafter=False, sampling=SMP)
        r.eng.set_state(dev([ctx]), dev([g]), dev(h[None], torch.float32), batch=1, ctx_bound=ctx)
        r.eng.step(dev(planted[None]), out)
        r.eng.poll()
        _, gaps = oracle_draws(ref["logits"], ref["packed"]["pos"], SMP, 0)
        if (gaps > GAP).all():
            a = ref["n_accept"]
            assert int(out.n_accept[0]) == a and int(out.best[0]) == ref["best"]
            assert out.tokens[0, :a + 1].tolist() == ref["emitted"]
            c_ctx, c_root, c_h = r.eng.get_state()
            assert int(c_ctx[0]) == ref["ctx"] and int(c_root[0]) == ref["g"]
            assert np.abs(c_h[0].cpu().numpy() - ref["h"]).max() < TOL_FP32
            checked += 1
        ctx, g, h = ref["ctx"], ref["g"], ref["h"]
        emitted.extend(ref["emitted"])
        accepted.append(ref["n_accept"])
    assert emitted == plain[:len(emitted)]                  # the oracle's own losslessness, on this workload
    assert checked >= 5 and max(accepted) >= 2
    r.eng.close()


@pytest.mark.parametrize("cfg", [None, BF16])
def test_speculative_stream_equals_plain_sampled_stream(cfg):
    """Free running on the GPU: with the same seed the speculative steps emit the tokens of plain sampled decoding
    (the paper's guarantee that the generated sequence is the LLM's own, carried over to temperature > 0)."""
    r = Rig(cfg=cfg) if cfg is not None else Rig()
    c = r.cfg
    L, BW = c["beam_length"], c["beam_width"]
    prompt = synth.make_prompts(c, 1)[0]
    steps = 24
    n_tok = 1 + steps * (L + 1)
    streams = {}
    for name, (T, seed) in dict(greedy=(0.0, 0), a=(1.0, 3), b=(1.0, 4)).items():
        r.eng.set_sampling(T, seed)
        r.eng.prefill([prompt])
        tok = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        _, root, _ = r.eng.get_state()
        s = [int(root[0])]
        for _ in range(n_tok - 1):
            r.eng.ar_step(tok)
            s.append(int(tok[0]))
        r.eng.poll()
        streams[name] = s
    assert streams["a"] != streams["greedy"] and streams["a"] != streams["b"]
    plain = streams["a"]
    r.eng.set_sampling(1.0, 3)
    r.eng.prefill([prompt])
    rng = np.random.default_rng(12)
    out = r.binding.AcceptOut(1, L, "cuda:0")
    spec, acc = [plain[0]], []
    for step in range(steps):
        planted = synth.plant_beams(plain[len(spec):len(spec) + L], BW, L, c["vocab"], rng, p=0.3)
        r.eng.step(dev(planted[None]), out)
        a = int(out.n_accept[0])
        spec.extend(out.tokens[0, :a + 1].tolist())
        acc.append(a)
        if spec != plain[:len(spec)]:
            break
    r.eng.poll()
    # the two streams come from differently batched launches of the same kernels: a near-tie of the perturbed scores
    # may split them; up to there they must agree, and a split this early would be a keying error
    agree = 0
    while agree < min(len(spec), len(plain)) and spec[agree] == plain[agree]:
        agree += 1
    assert agree >= min(len(spec), 40 if c["dtype"] == "fp32" else 12)
    assert np.mean(acc) > 1.0
    if c["dtype"] == "fp32":
        ar_ora, _, _ = ora.generate_ar(r.W, c, prompt, 24, c["max_ctx"], sampling=dict(temperature=1.0, seed=3))
        agree = 0
        while agree < 24 and ar_ora[agree] == plain[agree]:
            agree += 1
        assert agree >= 8
    r.eng.close()


def test_set_sampling_arguments_and_reset():
    from paper_2403_09919_b200.binding import RdError
    r = Rig()
    prompt = synth.make_prompts(r.cfg, 1)[0]
    r.eng.prefill([prompt])
    _, root0, _ = r.eng.get_state()
    for bad in (-1.0, float("nan"), float("inf")):
        with pytest.raises(RdError) as e:
            r.eng.set_sampling(bad, 1)
        assert e.value.code == 1
    r.eng.set_sampling(1.5, 9)
    r.eng.set_sampling(0.0, 9)                              # back to greedy
    r.eng.prefill([prompt])
    _, root1, _ = r.eng.get_state()
    r.eng.poll()
    assert int(root0[0]) == int(root1[0])
    r.eng.close()


def test_draw_frequencies_on_the_gpu_follow_the_softmax():
    """Distribution-level check through the CUDA path: the same verification pass under 600 seeds; for every packed
    row the counts of its eight likeliest tokens and of the rest against softmax(logits / T) of the logits the GPU
    returned (chi-square, 8 degrees of freedom, all rows pooled by their worst statistic)."""
    r = Rig()
    c = r.cfg
    T = 0.6
    prompt = synth.make_prompts(c, 1)[0]
    r.eng.prefill([prompt])                                   # greedy root: the same rows under every seed
    beams = np.random.default_rng(5).integers(0, 3, size=(1, c["beam_width"], c["beam_length"]))
    pk = r.eng.pack(dev(beams))
    n = int(pk.n[0])
    n_seeds = 600
    draws = np.zeros((n_seeds, n), dtype=np.int64)
    logits = None
    for seed in range(n_seeds):
        r.eng.set_sampling(T, 1000 + seed)
        toks, _, lg = r.eng.verify(pk, want_logits=logits is None)
        draws[seed] = toks[0, :n].cpu().numpy()
        if logits is None:
            logits = lg[0, :n].cpu().numpy().astype(np.float64)
    r.eng.poll()
    worst = 0.0
    for row in range(n):
        z = logits[row] / T
        p = np.exp(z - z.max())
        p /= p.sum()
        top = np.argsort(-p)[:8]
        expect = np.append(p[top], 1.0 - p[top].sum()) * n_seeds
        counts = np.array([(draws[:, row] == t).sum() for t in top] + [0])
        counts[-1] = n_seeds - counts[:-1].sum()
        worst = max(worst, float(((counts - expect) ** 2 / np.maximum(expect, 1e-9)).sum()))
    # P[chi2_8 > 40] is about 3e-6 per row; 17 rows at most
    assert worst < 40.0, worst
    # rows that choose the token of the same position share their noise: with equal logits they would agree; across
    # seeds the draws of one row do vary
    assert len(set(draws[:, 0].tolist())) > 3
    r.eng.close()

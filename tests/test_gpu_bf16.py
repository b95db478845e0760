"""Parity of the bf16 path (tcgen05 projections) with the oracle.

The oracle runs on the same bf16-rounded weight values in full precision, so the tolerance only
has to cover the rounding of activations to bf16 in front of every projection and in the KV cache:
logits within 3e-2 of the row's largest |logit|.  Decisions taken from floats (argmax, accepted
length) are compared where the oracle's top-2 gap exceeds twice that bound.
"""
import numpy as np
import pytest
import torch

from helpers import check_beams_within, dev, first_mismatch, Rig, tolerant_beam_search, top2_gap
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu

REL = 3e-2
EPS_SCORE = 2e-3     # drafter scores against the oracle with bf16 storage: measured 5.7e-4 (tests/test_gpu_drafter_beams.py)

# shapes that are NOT multiples of the 128 x 64 tiles: vocabulary 1000, d_ffn 1376
RAGGED = dict(synth.CONFIGS["tiny"], dtype="bf16", d_model=512, n_heads=4, d_ffn=1376, vocab=1000, d_rnn=512,
              max_ctx=400, beam_width=8, beam_length=5, prompt_len=96)


def rel_err(got, ref):
    scale = np.abs(ref).max(axis=-1, keepdims=True)
    return float((np.abs(got - ref) / scale).max())


def decided(ref_logits):
    """Rows whose argmax cannot be flipped by an error within the tolerance."""
    bound = REL * np.abs(ref_logits).max(axis=-1)
    return top2_gap(ref_logits) > np.maximum(0.05, 2 * bound)


def prefilled(rig, n=96, seed=0):
    prompt = np.random.default_rng(seed).integers(0, rig.cfg["vocab"], size=n)
    rig.eng.prefill([prompt])
    kv = rig.new_kv()
    ctx, g, h = ora.prefill(rig.W, rig.cfg, prompt, kv, rig.odt)
    return prompt, kv, ctx, g, h


def check_verify(rig, beams_alphabet=3):
    cfg = rig.cfg
    BW, L = cfg["beam_width"], cfg["beam_length"]
    prompt, kv, ctx, g, h = prefilled(rig)
    c_ctx, c_root, c_h = rig.eng.get_state()
    rig.eng.poll()
    assert int(c_ctx[0]) == ctx
    assert rel_err(c_h[0].cpu().numpy()[None], np.asarray(h)[None]) < REL
    # teacher-force the root/h so both sides verify the same packed rows
    rig.eng.set_state(None, dev([g]), dev(np.asarray(h, dtype=np.float32)[None], torch.float32))
    beams = np.random.default_rng(1).integers(0, beams_alphabet, size=(1, BW, L))
    pk = rig.eng.pack(dev(beams))
    argmax, hidden, logits = rig.eng.verify(pk, want_logits=True)
    rig.eng.poll()
    aug = np.concatenate([np.full((BW, 1), g), beams[0]], axis=1)
    p = ora.pack_beam(aug, ctx)
    n = p["n"]
    assert int(pk.n[0]) == n and pk.tokens[0, :n].tolist() == p["tokens"].tolist()
    rh, rl = ora.llm_forward(rig.W, cfg, p["tokens"], p["pos"], p["mask"], kv, ctx, rig.odt)
    got = logits[0, :n].cpu().numpy()
    assert rel_err(got, rl) < REL
    assert rel_err(hidden[0, :n].cpu().numpy(), rh) < REL
    sure = decided(rl)
    assert (argmax[0, :n].cpu().numpy()[sure] == rl.argmax(1)[sure]).all()
    return rel_err(got, rl)


def test_verify_ragged_shapes():
    check_verify(Rig(cfg=RAGGED))


def test_verify_7b_shapes_two_layers():
    check_verify(Rig(cfg=synth.with_layers(dict(synth.CONFIGS["7b"], max_ctx=256), 2), oracle_dtype=np.float32))


@pytest.mark.parametrize("vocab,d_ffn", [(1000, 1376), (1100, 1440)])
def test_tensor_core_path_matches_cuda_core_path(vocab, d_ffn):
    """The second shape gives the LM head 9 and the gate+up projection 23 weight tiles: odd counts, so the last
    pair of tiles of a stage has a tile that lies past the matrix."""
    from paper_2403_09919_b200 import binding
    outs = []
    for flags in (0, binding.RD_FLAG_FORCE_SIMT):
        r = Rig(cfg=dict(RAGGED, vocab=vocab, d_ffn=d_ffn), flags=flags)
        prompt = np.random.default_rng(0).integers(0, 1000, size=96)
        r.eng.prefill([prompt])
        beams = np.random.default_rng(1).integers(0, 3, size=(1, 8, 5))
        pk = r.eng.pack(dev(beams))
        am, hid, lg = r.eng.verify(pk, want_logits=True)
        r.eng.poll()
        outs.append((int(pk.n[0]), lg[0].cpu().numpy()))
        r.eng.close()
    n = outs[0][0]
    assert rel_err(outs[0][1][:n], outs[1][1][:n]) < 1e-2


def run_steps(rig, n_steps, seed, p=0.3, rho=0.3):
    """Teacher-forced steps through pack / verify / accept.  The LLM's greedy tokens are compared
    where the oracle's gap decides them; acceptance and compaction are checked bit-exactly against
    the oracle's rule applied to the GPU's own greedy tokens."""
    cfg = rig.cfg
    BW, L = cfg["beam_width"], cfg["beam_length"]
    prompt, kv, ctx, g, h = prefilled(rig)
    ar, _, _ = ora.generate_ar(rig.W, cfg, prompt, 2 + n_steps * (L + 1), cfg["max_ctx"], rig.odt)
    rng = np.random.default_rng(seed)
    emitted, full_match = [g], 0
    for step in range(n_steps):
        planted = synth.plant_beams(ar[len(emitted):len(emitted) + L], BW, L, cfg["vocab"], rng, p=p, rho=rho)
        ref = ora.spec_step(rig.W, rig.D, cfg, kv, ctx, g, h, BW, L, planted=planted, run_drafter=False, dtype=rig.odt)
        rig.eng.set_state(dev([ctx]), dev([g]), dev(np.asarray(h, dtype=np.float32)[None], torch.float32), batch=1,
                          ctx_bound=ctx)
        beams_d = dev(planted[None])
        pk = rig.eng.pack(beams_d)
        argmax, hidden, logits = rig.eng.verify(pk, want_logits=True)
        out = rig.eng.accept(beams_d, pk, argmax, hidden)
        rig.eng.poll()
        n = ref["packed"]["n"]
        assert int(pk.n[0]) == n and pk.unpack[0].cpu().numpy().tolist() == ref["packed"]["unpack"].tolist()
        assert rel_err(logits[0, :n].cpu().numpy(), ref["logits"]) < REL
        am = argmax[0, :n].cpu().numpy()
        sure = decided(ref["logits"])
        assert (am[sure] == ref["argmax"][sure]).all()
        a, best, toks = ora.accept_greedy(planted, ref["packed"]["unpack"], am)
        assert int(out.n_accept[0]) == a and int(out.best[0]) == best
        assert out.tokens[0, :a + 1].tolist() == toks and (out.tokens[0, a + 1:] == -1).all()
        c_ctx, c_root, c_h = rig.eng.get_state()
        assert int(c_ctx[0]) == ctx + 1 + a and int(c_root[0]) == toks[-1]
        if (am == ref["argmax"]).all():
            assert a == ref["n_accept"] and toks == ref["emitted"]
        if a == ref["n_accept"] and toks == ref["emitted"]:
            # same outcome as the oracle's step (rows off the accepted path may differ at near-ties): the handed-over
            # hidden state and the compacted cache must then agree too
            full_match += 1
            assert rel_err(c_h[0].cpu().numpy()[None], np.asarray(ref["h"])[None]) < REL
            kvg = rig.eng.kv_view()[:, 0, 0, :, :ref["ctx"]].float().cpu().numpy().transpose(0, 2, 1, 3)
            assert np.abs(kvg - kv.k[:, :ref["ctx"]]).max() < REL * np.abs(kv.k[:, :ref["ctx"]]).max()
        else:
            break                                     # an undecided row changed the outcome: stop here
        ctx, g, h = ref["ctx"], ref["g"], ref["h"]
        emitted.extend(ref["emitted"])
    return full_match


def test_step_teacher_forced_ragged():
    assert run_steps(Rig(cfg=RAGGED), 6, seed=2) >= 2


def test_draft_scores_ragged():
    rig = Rig(cfg=RAGGED)
    prompt, kv, ctx, g, h = prefilled(rig)
    rig.eng.set_state(None, dev([g]), dev(np.asarray(h, dtype=np.float32)[None], torch.float32))
    beams, scores = rig.eng.draft()
    rig.eng.poll()
    sc = scores[0].cpu().numpy()
    assert (np.diff(sc) <= 0).all()
    # each returned score is the drafter's log-probability of that sequence (within the bf16 bound)
    for b, s in zip(beams[0].cpu().numpy(), sc):
        assert abs(ora.sequence_logprob(rig.D, rig.W["tok_emb"], g, h, b, rig.odt) - s) < REL * abs(s)
    # the beams themselves, against the oracle with the path's bf16 storage and every decision widened by the score
    # error bound (tests/test_gpu_drafter_beams.py derives it): no certain beam missing, none that is ruled out
    sets = tolerant_beam_search(ora, rig.D, rig.W["tok_emb"], g, np.asarray(h, np.float32).astype(np.float64), 8, 5, EPS_SCORE, store="bf16")
    check_beams_within(sets, beams[0].cpu().numpy(), sc, EPS_SCORE)
    assert len(sets[0]) >= 4


def test_wide_beam_two_row_tiles():
    """Beam width 64 x length 5: up to 321 packed rows = two activation tiles per weight tile."""
    cfg = dict(RAGGED, beam_width=64, beam_length=5, max_ctx=500)
    rig = Rig(cfg=cfg)
    check_verify(rig, beams_alphabet=40)


def test_long_prompts_many_row_tiles():
    """Prompts of 700 and 450 tokens in one prefill of an engine sized for 16 sequences (passes of up to 656 rows: the
    first holds 656 rows of one sequence, the second its last 44 and the whole other prompt): three row tiles in the
    projections, the row-loop kernels, and 64-row causal attention tiles in which the warps' key ranges differ and
    start past the keys of an earlier pass.  The handed-over state (context length, last hidden vector) and a
    verification on top of the two caches must match the oracle."""
    # 16 heads of 64: 16 x 2 x 41 sixteen-row tiles would be several waves of CTAs, so the 64-row attention kernel runs
    cfg = dict(RAGGED, d_model=1024, n_heads=16, d_rnn=1024, max_batch=16, max_ctx=800)
    rig = Rig(cfg=cfg)
    rng = np.random.default_rng(11)
    prompts = [rng.integers(0, 1000, size=700), rng.integers(0, 1000, size=450)]
    rig.eng.prefill(prompts)
    rig.eng.poll()
    c_ctx, c_root, c_h = rig.eng.get_state()
    refs = []
    for b, pr in enumerate(prompts):
        kv = rig.new_kv()
        ctx, g, h = ora.prefill(rig.W, cfg, pr, kv)
        assert int(c_ctx[b]) == ctx
        assert rel_err(c_h[b].cpu().numpy()[None], np.asarray(h)[None]) < REL
        refs.append((kv, ctx, g, h))
    roots = np.array([r[2] for r in refs])
    hs = np.stack([np.asarray(r[3]) for r in refs]).astype(np.float32)
    rig.eng.set_state(None, dev(roots), dev(hs, torch.float32))
    beams = rng.integers(0, 4, size=(2, 8, 5))
    pk = rig.eng.pack(dev(beams))
    argmax, hidden, logits = rig.eng.verify(pk, want_logits=True)
    rig.eng.poll()
    for b, (kv, ctx, g, h) in enumerate(refs):
        aug = np.concatenate([np.full((8, 1), g), beams[b]], axis=1)
        p = ora.pack_beam(aug, ctx)
        n = p["n"]
        assert int(pk.n[b]) == n
        rh, rl = ora.llm_forward(rig.W, cfg, p["tokens"], p["pos"], p["mask"], kv, ctx)
        assert rel_err(logits[b, :n].cpu().numpy(), rl) < REL
        sure = decided(rl)
        assert (argmax[b, :n].cpu().numpy()[sure] == rl.argmax(1)[sure]).all()


def test_wide_beam_whose_rows_fit_one_tile_after_all():
    """Beam width 64 with heavily shared prefixes: the host-side bound is 321 rows (two row tiles), the packed rows are
    about 170, so the projections run a single tile and their consumers take the single-tile path of a launch that was
    laid out for two."""
    cfg = dict(RAGGED, beam_width=64, beam_length=5, max_ctx=500)
    rig = Rig(cfg=cfg)
    check_verify(rig, beams_alphabet=3)


def test_long_prompts_head_dim_128():
    """Four prompts (700, 300, 120 and 40 tokens) at head dimension 128 in an engine sized for 16 sequences: passes of up
    to 656 rows.  The long sequence's first pass takes the tensor-core (tcgen05) attention kernel -- 128-row causal
    tiles, the last one partly filled, chunks of 128 keys of which the last lies partly beyond every row's extent, tiles
    of the other sequences without rows; later passes run on top of the cache the first wrote.  State and a verification
    on top of it must match the oracle for every sequence."""
    cfg = dict(RAGGED, max_batch=16, max_ctx=800)   # d_model 512, 4 heads of 128
    rig = Rig(cfg=cfg)
    rng = np.random.default_rng(12)
    prompts = [rng.integers(0, 1000, size=n) for n in (700, 300, 120, 40)]
    rig.eng.prefill(prompts)
    rig.eng.poll()
    c_ctx, c_root, c_h = rig.eng.get_state()
    refs = []
    for b, pr in enumerate(prompts):
        kv = rig.new_kv()
        ctx, g, h = ora.prefill(rig.W, cfg, pr, kv)
        assert int(c_ctx[b]) == ctx
        assert rel_err(c_h[b].cpu().numpy()[None], np.asarray(h)[None]) < REL
        refs.append((kv, ctx, g, h))
    roots = np.array([r[2] for r in refs])
    hs = np.stack([np.asarray(r[3]) for r in refs]).astype(np.float32)
    rig.eng.set_state(None, dev(roots), dev(hs, torch.float32))
    beams = rng.integers(0, 4, size=(4, 8, 5))
    pk = rig.eng.pack(dev(beams))
    argmax, hidden, logits = rig.eng.verify(pk, want_logits=True)
    rig.eng.poll()
    for b, (kv, ctx, g, h) in enumerate(refs):
        aug = np.concatenate([np.full((8, 1), g), beams[b]], axis=1)
        p = ora.pack_beam(aug, ctx)
        n = p["n"]
        assert int(pk.n[b]) == n
        rh, rl = ora.llm_forward(rig.W, cfg, p["tokens"], p["pos"], p["mask"], kv, ctx)
        assert rel_err(logits[b, :n].cpu().numpy(), rl) < REL
        sure = decided(rl)
        assert (argmax[b, :n].cpu().numpy()[sure] == rl.argmax(1)[sure]).all()


def test_batched_ragged_many_rows():
    """Batch 16 x beam width 16: up to 1296 compact rows, six activation tiles, per-sequence contexts."""
    cfg = dict(RAGGED, max_batch=16, beam_width=16, beam_length=5, max_ctx=260)
    rig = Rig(cfg=cfg)
    rng = np.random.default_rng(3)
    prompts = [rng.integers(0, 1000, size=int(n)) for n in rng.integers(20, 150, size=16)]
    rig.eng.prefill(prompts)
    c_ctx, c_root, c_h = rig.eng.get_state()
    beams = rng.integers(0, 30, size=(16, 16, 5))
    refs = []
    for b, pr in enumerate(prompts):
        kv = rig.new_kv()
        ctx, g, h = ora.prefill(rig.W, cfg, pr, kv)
        assert int(c_ctx[b]) == ctx
        assert rel_err(c_h[b].cpu().numpy()[None], h[None]) < REL
        refs.append((kv, ctx, g, h))
    roots = np.array([r[2] for r in refs])
    hs = np.stack([r[3] for r in refs]).astype(np.float32)
    rig.eng.set_state(None, dev(roots), dev(hs, torch.float32))
    pk = rig.eng.pack(dev(beams))
    argmax, hidden, logits = rig.eng.verify(pk, want_logits=True)
    rig.eng.poll()
    assert int(pk.n.sum()) > 512
    for b, (kv, ctx, g, h) in enumerate(refs):
        aug = np.concatenate([np.full((16, 1), g), beams[b]], axis=1)
        p = ora.pack_beam(aug, ctx)
        n = p["n"]
        assert int(pk.n[b]) == n
        rh, rl = ora.llm_forward(rig.W, cfg, p["tokens"], p["pos"], p["mask"], kv, ctx)
        assert rel_err(logits[b, :n].cpu().numpy(), rl) < REL
        sure = decided(rl)
        assert (argmax[b, :n].cpu().numpy()[sure] == rl.argmax(1)[sure]).all()


def test_free_running_lossless_up_to_the_first_near_tie():
    """Lossless property, free running on the bf16 kernels: both the GPU's autoregressive stream and
    its planted-beam speculative stream reproduce the oracle's greedy stream for as long as the
    oracle's top-2 logit gap exceeds 0.05 at every token (the two GPU paths sum in different orders,
    so beyond a near-tie they may legitimately part), and accepted lengths follow the closed form."""
    rig = Rig(cfg=RAGGED)
    cfg = rig.cfg
    BW, L = cfg["beam_width"], cfg["beam_length"]
    n_tok = 48
    best = None
    for seed in range(4, 40):                      # the first prompt whose greedy stream stays decided for a while
        prompt = np.random.default_rng(seed).integers(0, 1000, size=64)
        kv = rig.new_kv()
        ctx, g, h = ora.prefill(rig.W, cfg, prompt, kv)
        ref, decisive = [g], None
        for i in range(n_tok + L):
            g, h, logits = ora.ar_step(rig.W, cfg, kv, ctx, g)
            ctx += 1
            if decisive is None and top2_gap(logits) <= 0.05:
                decisive = len(ref)                # ref[:decisive] are decided, the next token is a near-tie
            ref.append(g)
        decisive = len(ref) - L if decisive is None else min(decisive, len(ref) - L)
        if decisive >= 18:
            best = (prompt, ref, decisive)
            break
    assert best is not None
    prompt, ref, decisive = best
    rig.eng.prefill([prompt])
    tok = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    ar = [int(rig.eng.get_state()[1][0])]
    for _ in range(decisive - 1):
        rig.eng.ar_step(tok)
        ar.append(int(tok[0]))
    assert ar == ref[:decisive]
    rig.eng.prefill([prompt])
    rng = np.random.default_rng(5)
    out = rig.binding.AcceptOut(1, L, "cuda:0")
    spec = [int(rig.eng.get_state()[1][0])]
    steps = 0
    while len(spec) + L + 1 <= decisive:
        planted = synth.plant_beams(ref[len(spec):len(spec) + L], BW, L, cfg["vocab"], rng, p=0.3, rho=0.3)
        rig.eng.step(dev(planted[None]), out)
        a = int(out.n_accept[0])
        assert a == first_mismatch(planted, ref[len(spec):len(spec) + L]).max()
        spec.extend(out.tokens[0, :a + 1].tolist())
        steps += 1
    rig.eng.poll()
    assert steps >= 2 and spec == ref[:len(spec)]


def _rig_with_env(env, **kw):
    import os
    old = {k: os.environ.get(k) for k in env}
    os.environ.update(env)
    try:
        return Rig(**kw)
    finally:
        for k, v in old.items():
            if v is None:
                del os.environ[k]
            else:
                os.environ[k] = v


@pytest.mark.parametrize("bw,batch,prompt", [(8, 1, 96), (16, 3, 300), (32, 2, 700)])
def test_projection_on_cta_pairs_matches_the_one_cta_kernel(bw, batch, prompt):
    """The CTA-pair projection (two CTAs share one MMA: each loads its weight tile and half of the activation box)
    against the one-CTA kernel on the same weights and inputs: one row tile of 48 rows, one of 243 rows at most, and
    several row tiles with a prompt processed in one pass of three; shapes that are not multiples of the tiles (an odd
    number of weight tiles leaves the pair's second tile past the matrix).  Both sum each output element over the same
    k-blocks in fp32, only the grouping into partial sums differs; a last-bit difference becomes a bf16 step (2^-9)
    where an activation is rounded in front of the next projection, hence the same bound as between the tensor-core
    and the CUDA-core path."""
    cfg = dict(RAGGED, vocab=1100, d_ffn=1440, beam_width=bw, max_batch=batch, max_ctx=prompt + 200)
    outs = []
    roots = None
    for env in (dict(RD_TC_CTA2_MIN="17", RD_TC_CTA2_PREFILL="1"), dict(RD_TC_CTA2="0")):
        r = _rig_with_env(env, cfg=cfg)
        rng = np.random.default_rng(0)
        prompts = [rng.integers(0, cfg["vocab"], size=prompt - 7 * b) for b in range(batch)]
        r.eng.prefill(prompts)
        # both engines verify the same root tokens (the first engine's: a near-tie in the root's logits may fall either way)
        if roots is None:
            roots = r.eng.get_state()[1].clone()
        r.eng.set_state(None, roots, None)
        beams = np.random.default_rng(1).integers(0, 3, size=(batch, bw, 5))
        pk = r.eng.pack(dev(beams))
        am, hid, lg = r.eng.verify(pk, want_logits=True)
        r.eng.poll()
        outs.append((pk.n.cpu().numpy(), lg.cpu().numpy(), r.eng.get_state()[2].cpu().numpy()))
        r.eng.close()
    assert (outs[0][0] == outs[1][0]).all()
    for b in range(batch):
        n = int(outs[0][0][b])
        assert rel_err(outs[0][1][b, :n], outs[1][1][b, :n]) < 1e-2
    assert rel_err(outs[0][2], outs[1][2]) < 1e-2


@pytest.mark.parametrize("bw", [33, 64])
def test_draft_scores_wide_beams(bw):
    """Beam widths above 32 through the two-kernel selection (segments of the vocabulary, then one merging CTA per
    surviving beam ranking BW x BW candidates): scores sorted, every score the log-probability of its sequence, best
    score and total mass as the oracle's, identical beams where the oracle's candidate gaps are clear of the bound."""
    cfg = dict(RAGGED, beam_width=bw, max_ctx=96 + 2 + bw * 5 + 8)
    rig = Rig(cfg=cfg)
    prompt, kv, ctx, g, h = prefilled(rig)
    rig.eng.set_state(None, dev([g]), dev(np.asarray(h, dtype=np.float32)[None], torch.float32))
    beams, scores = rig.eng.draft()
    rig.eng.poll()
    sc = scores[0].cpu().numpy()
    bm = beams[0].cpu().numpy()
    assert (np.diff(sc) <= 0).all()
    assert len({tuple(b) for b in bm.tolist()}) == bw                      # distinct sequences
    for i in (0, 1, bw // 2, bw - 1):
        assert abs(ora.sequence_logprob(rig.D, rig.W["tok_emb"], g, h, bm[i], rig.odt) - sc[i]) < REL * abs(sc[i])
    sets = tolerant_beam_search(ora, rig.D, rig.W["tok_emb"], g, np.asarray(h, np.float32).astype(np.float64), bw, 5, EPS_SCORE, store="bf16")
    check_beams_within(sets, bm, sc, EPS_SCORE)
    assert len(sets[0]) >= bw // 2
    rig.eng.close()

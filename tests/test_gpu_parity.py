"""Parity of the CUDA path (through the C ABI) with the oracle, tiny fp32 configuration.

Integer outputs are compared bit-exactly.  Where a float decides an integer (argmax, top-k) the
comparison is made only where the oracle's gap exceeds GAP; logits must agree within 2e-3.
"""
import numpy as np
import pytest
import torch

from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu

GAP = 0.05
TOL_FP32 = 2e-3
EPS_SCORE = 2e-5     # fp32 drafter scores against the fp64 oracle: measured 3e-6 at scores of about -25


from helpers import check_beams_within, dev, first_mismatch, Rig, tolerant_beam_search, top2_gap  # noqa: E402


@pytest.fixture(scope="module")
def rig():
    return Rig()


# ------------------------------------------------------------------ pack
def check_pack(eng, beams, roots, ctxs, tree=True):
    B, BW, L = beams.shape
    eng.set_state(dev(ctxs), dev(roots), None, batch=B, ctx_bound=int(max(ctxs)))
    pk = eng.pack(dev(beams))
    eng.poll()
    nmax = 1 + BW * L
    for b in range(B):
        aug = np.concatenate([np.full((BW, 1), roots[b]), beams[b]], axis=1)
        ref = ora.pack_beam(aug, int(ctxs[b])) if tree else ora.flat_beam(aug, int(ctxs[b]))
        n = int(pk.n[b])
        assert n == ref["n"]
        assert pk.tokens[b, :n].tolist() == ref["tokens"].tolist()
        assert pk.unpack[b].cpu().numpy().tolist() == ref["unpack"].tolist()
        assert pk.pos[b, :n].tolist() == ref["pos"].tolist()
        assert pk.parent[b, :n].tolist() == ref["parent"].tolist()
        assert (pk.mask_bool(b) == ref["mask"]).all()
        # padding rows have defined values
        assert (pk.tokens[b, n:] == 0).all() and (pk.pos[b, n:] == 0).all() and (pk.parent[b, n:] == -1).all()
        assert (pk.mask[b, n:] == 0).all()
    return pk


def test_pack_paper_example_and_edges(rig):
    eng = rig.eng
    beam = np.array([[[91, 92, 93, 95], [91, 92, 94, 96], [91, 92, 93, 97], [91, 92, 93, 97]]])   # + a duplicate row
    pk = check_pack(eng, beam, [7], [100])
    assert pk.tokens[0, :8].tolist() == [7, 91, 92, 93, 95, 94, 96, 97]
    same = np.tile(np.array([[[1, 2, 3, 4]]]), (1, 4, 1))
    assert int(check_pack(eng, same, [0], [5]).n[0]) == 5
    distinct = (np.arange(4)[:, None] * 10 + np.arange(4)[None, :])[None]
    assert int(check_pack(eng, distinct, [1023], [5]).n[0]) == 17
    edge = np.array([[[0, 1023, 0, 1023], [0, 1023, 0, 0], [1023, 0, 0, 0], [0, 0, 0, 0]]])
    check_pack(eng, edge, [0], [64])


def test_pack_random_wide_and_batched():
    rng = np.random.default_rng(3)
    for (B, BW, L, v) in ((1, 64, 5, 3), (4, 16, 5, 2), (3, 1, 4, 5), (2, 32, 5, 4), (1, 8, 5, 2)):
        r = Rig(max_batch=B, beam_width=BW, beam_length=L, max_ctx=600)
        for trial in range(4):
            beams = rng.integers(0, v, size=(B, BW, L))
            check_pack(r.eng, beams, rng.integers(0, 1024, size=B), rng.integers(1, 200, size=B))
        r.eng.close()


def test_pack_no_tree_flag():
    from paper_2403_09919_b200 import binding
    r = Rig(flags=binding.RD_FLAG_NO_TREE)
    beams = np.random.default_rng(4).integers(0, 2, size=(1, 4, 4))
    pk = check_pack(r.eng, beams, [3], [10], tree=False)
    assert int(pk.n[0]) == 17


# ------------------------------------------------------------------ prefill, verify, draft
def prefilled(rig, prompt=None):
    prompt = synth.make_prompts(rig.cfg, 1)[0] if prompt is None else prompt
    rig.eng.prefill([prompt])
    kv = rig.new_kv()
    ctx, g, h = ora.prefill(rig.W, rig.cfg, prompt, kv)
    return prompt, kv, ctx, g, h


def test_prefill_state(rig):
    prompt, kv, ctx, g, h = prefilled(rig)
    c_ctx, c_root, c_h = rig.eng.get_state()
    rig.eng.poll()
    assert int(c_ctx[0]) == ctx
    assert np.abs(c_h[0].cpu().numpy() - h).max() < TOL_FP32
    assert int(c_root[0]) == g
    kvg = rig.eng.kv_view()[:, :, 0, :, :ctx].cpu().numpy()              # [layers, 2, H, ctx, hd]
    assert np.abs(kvg[:, 0].transpose(0, 2, 1, 3) - kv.k[:, :ctx]).max() < TOL_FP32
    assert np.abs(kvg[:, 1].transpose(0, 2, 1, 3) - kv.v[:, :ctx]).max() < TOL_FP32


def test_prefill_in_several_passes():
    # a prompt longer than one forward pass (256 rows) exercises the chunked causal path
    r = Rig(max_ctx=700)
    prompt = np.random.default_rng(5).integers(0, 1024, size=600)
    _, kv, ctx, g, h = prefilled(r, prompt)
    c_ctx, c_root, c_h = r.eng.get_state()
    assert int(c_ctx[0]) == 600 and np.abs(c_h[0].cpu().numpy() - h).max() < TOL_FP32


def test_verify_logits_and_argmax(rig):
    prompt, kv, ctx, g, h = prefilled(rig)
    rng = np.random.default_rng(6)
    beams = rng.integers(0, 3, size=(1, 4, 4))
    pk = rig.eng.pack(dev(beams))
    argmax, hidden, logits = rig.eng.verify(pk, want_logits=True)
    rig.eng.poll()
    aug = np.concatenate([np.full((4, 1), g), beams[0]], axis=1)
    p = ora.pack_beam(aug, ctx)
    rh, rl = ora.llm_forward(rig.W, rig.cfg, p["tokens"], p["pos"], p["mask"], kv, ctx)
    n = p["n"]
    assert np.abs(logits[0, :n].cpu().numpy() - rl).max() < TOL_FP32
    assert np.abs(hidden[0, :n].cpu().numpy() - rh).max() < TOL_FP32
    sure = top2_gap(rl) > GAP
    assert (argmax[0, :n].cpu().numpy()[sure] == rl.argmax(1)[sure]).all()
    assert (argmax[0, n:] == -1).all()
    # provisional K/V rows are in the cache at slots ctx + n
    kvg = rig.eng.kv_view()[:, 0, 0, :, ctx:ctx + n].cpu().numpy().transpose(0, 2, 1, 3)
    assert np.abs(kvg - kv.k[:, ctx:ctx + n]).max() < TOL_FP32


def test_draft_beams_and_scores(rig):
    prompt, kv, ctx, g, h = prefilled(rig)
    beams, scores = rig.eng.draft()
    rig.eng.poll()
    # the oracle's beam search with every decision widened by the fp32 error bound: for this state no decision comes
    # within it (an oracle-side fact, asserted), so the beams must be the oracle's element by element
    sets = tolerant_beam_search(ora, rig.D, rig.W["tok_emb"], g, h, 4, 4, EPS_SCORE)
    assert len(sets[0]) == 4 and not sets[1] and sets[2] == 0
    assert check_beams_within(sets, beams[0].cpu().numpy(), scores[0].cpu().numpy(), EPS_SCORE) == 4
    rb, rs = ora.beam_search(rig.D, rig.W["tok_emb"], g, h, 4, 4)
    assert beams[0].cpu().numpy().tolist() == rb.tolist()
    assert np.abs(scores[0].cpu().numpy() - rs).max() < EPS_SCORE
    assert (np.diff(scores[0].cpu().numpy()) <= 0).all()
    # whatever the ties, each returned score is the drafter's log-probability of that sequence
    for b, s in zip(beams[0].cpu().numpy(), scores[0].cpu().numpy()):
        assert abs(ora.sequence_logprob(rig.D, rig.W["tok_emb"], g, h, b) - s) < TOL_FP32


def test_draft_beam_width_one():
    r = Rig(beam_width=1)
    prompt, kv, ctx, g, h = prefilled(r)
    beams, scores = r.eng.draft()
    rb, rs = ora.beam_search(r.D, r.W["tok_emb"], g, h, 1, 4)
    assert abs(float(scores[0, 0]) - ora.sequence_logprob(r.D, r.W["tok_emb"], g, h, beams[0, 0].cpu().numpy())) < TOL_FP32
    assert abs(float(scores[0, 0]) - rs[0]) < TOL_FP32


# ------------------------------------------------------------------ whole step, teacher-forced
def run_steps(rig, n_steps, p, rho, seed, drafted=False):
    cfg = rig.cfg
    BW, L = cfg["beam_width"], cfg["beam_length"]
    prompt, kv, ctx, g, h = prefilled(rig)
    ar, _, _ = ora.generate_ar(rig.W, cfg, prompt, 2 + n_steps * (L + 1), cfg["max_ctx"])
    rng = np.random.default_rng(seed)
    out = rig.binding.AcceptOut(1, L, "cuda:0")
    emitted = [g]
    accepted = []
    drafted_equal = []
    for step in range(n_steps):
        planted = None if drafted else synth.plant_beams(ar[len(emitted):len(emitted) + L], BW, L, cfg["vocab"], rng, p=p, rho=rho)
        ref = ora.spec_step(rig.W, rig.D, cfg, kv, ctx, g, h, BW, L, planted=planted, run_drafter=drafted)
        # teacher forcing: both sides start the step from the oracle's state
        rig.eng.set_state(dev([ctx]), dev([g]), dev(h[None], torch.float32), batch=1, ctx_bound=ctx)
        if drafted:
            gb, gs = rig.eng.draft()
            sets = tolerant_beam_search(ora, rig.D, rig.W["tok_emb"], g, h, BW, L, EPS_SCORE)
            check_beams_within(sets, gb[0].cpu().numpy(), gs[0].cpu().numpy(), EPS_SCORE)
            if not sets[1]:
                # no decision within the error bound: the drafter's beams are the oracle's, and the step runs on them
                assert gb[0].cpu().numpy().tolist() == ref["beams"].tolist()
                drafted_equal.append(step)
                rig.eng.step(None, out)
            else:
                rig.eng.step(dev(ref["beams"][None]), out)   # a near-tie: both sides verify the oracle's beams
        else:
            rig.eng.step(dev(planted[None]), out)
        rig.eng.poll()
        if (top2_gap(ref["logits"]) > GAP).all():
            assert int(out.n_accept[0]) == ref["n_accept"]
            assert int(out.best[0]) == ref["best"]
            a = ref["n_accept"]
            assert out.tokens[0, :a + 1].tolist() == ref["emitted"]
            assert (out.tokens[0, a + 1:] == -1).all()
        elif int(out.n_accept[0]) != ref["n_accept"]:
            break
        ctx, g, h = ref["ctx"], ref["g"], ref["h"]
        c_ctx, c_root, c_h = rig.eng.get_state()
        assert int(c_ctx[0]) == ctx and int(c_root[0]) == g
        assert np.abs(c_h[0].cpu().numpy() - h).max() < TOL_FP32
        emitted.extend(ref["emitted"])
        accepted.append(ref["n_accept"])
        # compaction: the cache up to the new context equals the oracle's
        kvg = rig.eng.kv_view()[:, :, 0, :, :ctx].cpu().numpy()
        assert np.abs(kvg[:, 0].transpose(0, 2, 1, 3) - kv.k[:, :ctx]).max() < TOL_FP32
        assert np.abs(kvg[:, 1].transpose(0, 2, 1, 3) - kv.v[:, :ctx]).max() < TOL_FP32
    assert emitted == ar[:len(emitted)]
    if drafted:
        return accepted, drafted_equal
    return accepted


def test_step_planted_teacher_forced(rig):
    acc = run_steps(rig, 12, 0.3, 0.0, seed=7)
    assert len(acc) >= 8 and max(acc) >= 2


def test_step_planted_with_shared_prefixes(rig):
    acc = run_steps(rig, 8, 0.3, 0.5, seed=8)
    assert len(acc) >= 6


def test_step_all_accepted_and_none_accepted(rig):
    assert set(run_steps(rig, 3, 0.0, 0.0, seed=9)) == {4}        # a = L
    assert set(run_steps(rig, 3, 1.0, 0.0, seed=10)) == {0}       # a = 0: only the bonus


def test_step_with_drafted_beams(rig):
    """Whole steps on the drafter's own beams (no planted input): in at least three of the four steps the GPU's beams
    equal the oracle's element by element and the step's outcome is compared on them."""
    accepted, drafted_equal = run_steps(rig, 4, 0.0, 0.0, seed=11, drafted=True)
    assert len(accepted) == 4 and len(drafted_equal) >= 3


def test_full_tiny_config_32_steps_lossless_free_running(rig):
    """32 decode steps of the tiny workload, free running on the GPU: the speculative stream equals
    the GPU's own autoregressive stream (same kernels) and, where the oracle's gaps allow, the oracle's."""
    cfg = rig.cfg
    L, BW = cfg["beam_length"], cfg["beam_width"]
    prompt = synth.make_prompts(cfg, 1)[0]
    n_tok = 1 + 32 * (L + 1)
    rig.eng.prefill([prompt])
    tok = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    _, root, _ = rig.eng.get_state()
    ar_gpu = [int(root[0])]
    for _ in range(n_tok - 1):
        rig.eng.ar_step(tok)
        ar_gpu.append(int(tok[0]))
    rig.eng.poll()
    rig.eng.prefill([prompt])
    rng = np.random.default_rng(12)
    out = rig.binding.AcceptOut(1, L, "cuda:0")
    spec = [ar_gpu[0]]
    acc = []
    for step in range(32):
        planted = synth.plant_beams(ar_gpu[len(spec):len(spec) + L], BW, L, cfg["vocab"], rng, p=0.3)
        rig.eng.step(dev(planted[None]), out)
        a = int(out.n_accept[0])
        assert a == first_mismatch(planted, ar_gpu[len(spec):len(spec) + L]).max()
        spec.extend(out.tokens[0, :a + 1].tolist())
        acc.append(a)
    rig.eng.poll()
    assert spec == ar_gpu[:len(spec)]
    assert np.mean(acc) > 1.0
    ar_ora, _, _ = ora.generate_ar(rig.W, cfg, prompt, 40, cfg["max_ctx"])
    agree = 0
    while agree < 40 and ar_ora[agree] == ar_gpu[agree]:
        agree += 1
    assert agree >= 8            # near-ties (gap < 1e-4) may eventually split the two streams


# ------------------------------------------------------------------ batch, errors
def test_batched_ragged_step():
    r = Rig(max_batch=3, max_ctx=200)
    cfg = r.cfg
    rng = np.random.default_rng(13)
    prompts = [rng.integers(0, 1024, size=n) for n in (20, 64, 37)]
    r.eng.prefill(prompts)
    states, beams = [], []
    for b, p in enumerate(prompts):
        kv = r.new_kv()
        ctx, g, h = ora.prefill(r.W, cfg, p, kv)
        ar, _, _ = ora.generate_ar(r.W, cfg, p, 6, cfg["max_ctx"])
        beams.append(synth.plant_beams(ar[1:5], 4, 4, 1024, rng, p=0.3, rho=0.3))
        states.append((kv, ctx, g, h))
    c_ctx, c_root, c_h = r.eng.get_state()
    for b, (kv, ctx, g, h) in enumerate(states):
        assert int(c_ctx[b]) == ctx and int(c_root[b]) == g
        assert np.abs(c_h[b].cpu().numpy() - h).max() < TOL_FP32
    out = r.binding.AcceptOut(3, 4, "cuda:0")
    r.eng.step(dev(np.stack(beams)), out)
    r.eng.poll()
    c_ctx, c_root, c_h = r.eng.get_state()
    for b, (kv, ctx, g, h) in enumerate(states):
        ref = ora.spec_step(r.W, r.D, cfg, kv, ctx, g, h, 4, 4, planted=beams[b], run_drafter=False)
        if (top2_gap(ref["logits"]) > GAP).all():
            assert int(out.n_accept[b]) == ref["n_accept"] and int(out.best[b]) == ref["best"]
            assert out.tokens[b, :ref["n_accept"] + 1].tolist() == ref["emitted"]
            assert int(c_ctx[b]) == ref["ctx"] and int(c_root[b]) == ref["g"]
            assert np.abs(c_h[b].cpu().numpy() - ref["h"]).max() < TOL_FP32
            kvg = r.eng.kv_view()[:, 0, b, :, :ref["ctx"]].cpu().numpy().transpose(0, 2, 1, 3)
            assert np.abs(kvg - kv.k[:, :ref["ctx"]]).max() < TOL_FP32


def test_context_bound_follows_the_real_context():
    """The handle's host-side context bound grows by 1 + L per step, the most a step can accept; copies of the real
    context lengths that arrive later pull it back.  Here 48 steps accept about one token each: without the feedback
    the bound would pass 16 + 48 * 5 = 256 and the capacity check would refuse a step long before the cache is full."""
    cfg = dict(synth.CONFIGS["tiny"], max_ctx=16 + 48 * 2 + 17 + 10 * 5)
    r = Rig(cfg=cfg)
    r.eng.prefill([np.random.default_rng(14).integers(0, 1024, size=16)])
    out = r.binding.AcceptOut(1, 4, "cuda:0")
    rng = np.random.default_rng(15)
    for step in range(48):
        r.eng.step(dev(rng.integers(0, 1024, size=(1, 4, 4))), out)     # random candidates: at most a lucky token accepted
        if step % 8 == 7:
            r.eng.poll()                                                  # a serving loop reads its results now and then
    ctx = int(r.eng.get_state()[0][0])
    assert 16 + 48 <= ctx <= 16 + 48 * 2
    r.eng.close()


def test_errors(rig):
    from paper_2403_09919_b200.binding import RdError, ReDrafter
    eng = ReDrafter(rig.cfg, rig.w)
    with pytest.raises(RdError) as e:
        eng.step()
    assert e.value.code == 4                                   # no state yet
    with pytest.raises(RdError) as e:
        eng.prefill([np.zeros(rig.cfg["max_ctx"] - 3, dtype=np.int64)])
    assert e.value.code == 3                                   # no room for a step
    eng.prefill([np.array([1, 2, 3])])
    eng.set_state(ctx_bound=rig.cfg["max_ctx"] - 16)           # one step short of the capacity
    with pytest.raises(RdError) as e:
        eng.step()
    assert e.value.code == 3
    eng.set_state(ctx_bound=3)
    eng.set_state(None, dev([5000]), None)                     # a root token outside the vocabulary
    eng.step()
    with pytest.raises(RdError):
        eng.poll()
    eng.poll()                                                  # the status word was cleared
    with pytest.raises(RdError) as e:
        ReDrafter(dict(rig.cfg, beam_width=2000), rig.w)
    assert e.value.code == 2

"""Parity at the benchmark's own size: the 7B workload at its full depth (32 layers), beam width 8, beam length 5,
batch 1, in the launch configuration `bench.py` times (tensor-core projections, counter hand-off, tree attention).

The oracle (fp32 numpy on the same bf16-rounded weight values) needs about 13 GFLOP per row at this depth, so the
case keeps the prompt to 32 tokens and checks ONE step: the state after the prompt, the drafter's scores for sampled
beams, packing bit-exact, the verification logits of every packed row within the bf16 bound, greedy tokens where
the oracle's gap decides them, and acceptance + hand-off bit-exact against the oracle's rule applied to the GPU's
own greedy tokens.  The beams of the verified step are planted from the GPU's own autoregressive continuation (an
input recipe, not an expected value), so that several tokens are accepted.

Tolerance.  The bf16 path rounds every projection input and the KV cache to bf16 (relative step 2^-8); the oracle
does not.  That rounding noise is independent from layer to layer and, with random-init weights, is neither damped
nor amplified much on its way up, so it grows as the square root of the depth: measured relative L2 error of the
logits at this shape 0.8e-2 (1 layer), 1.1e-2 (2), 1.5e-2 (4), 2.0e-2 (8), 2.9e-2 (16), 4.1e-2 (32), i.e.
0.8e-2 x sqrt(depth); the worst row's max |error| / max |logit| is 1.5e-2 at two layers and 4.8e-2 at 32.  The
3e-2 bound of the depth-reduced parity cases therefore becomes 0.8e-2 x sqrt(32) x 1.5 = 7e-2 here.
"""
import numpy as np
import pytest
import torch

from helpers import Rig, dev, top2_gap
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu

REL = 7e-2   # 0.8e-2 x sqrt(32 layers) x 1.5: see the module docstring


def rel_err(got, ref):
    return float((np.abs(got - ref) / np.abs(ref).max(axis=-1, keepdims=True)).max())


def decided(ref_logits):
    bound = REL * np.abs(ref_logits).max(axis=-1)
    return top2_gap(ref_logits) > np.maximum(0.05, 2 * bound)


def test_one_step_of_the_7b_workload_at_full_depth():
    cfg = dict(synth.CONFIGS["7b"], max_ctx=256)
    rig = Rig(cfg=cfg, oracle_dtype=np.float32)
    BW, L = cfg["beam_width"], cfg["beam_length"]
    assert cfg["n_layers"] == 32 and BW == 8 and L == 5
    prompt = np.random.default_rng(40).integers(0, cfg["vocab"], size=32)

    # the GPU's own continuation, to plant beams from
    rig.eng.prefill([prompt])
    tok = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    cont = []
    for _ in range(L):
        rig.eng.ar_step(tok)
        cont.append(int(tok[0]))
    rig.eng.poll()

    # state after the prompt
    rig.eng.prefill([prompt])
    kv = rig.new_kv()
    ctx, g, h = ora.prefill(rig.W, cfg, prompt, kv, rig.odt)
    c_ctx, c_root, c_h = rig.eng.get_state()
    rig.eng.poll()
    assert int(c_ctx[0]) == ctx == 32
    assert rel_err(c_h[0].cpu().numpy()[None], np.asarray(h)[None]) < REL
    logits_last = np.asarray(h, dtype=np.float64) @ np.asarray(rig.W["lm_head"], dtype=np.float64).T
    if decided(logits_last[None])[0]:
        assert int(c_root[0]) == g

    # both sides continue from the oracle's state
    rig.eng.set_state(None, dev([g]), dev(np.asarray(h, dtype=np.float32)[None], torch.float32))

    # drafter: scores sorted, and the scores of sampled beams are those sequences' log-probabilities
    beams, scores = rig.eng.draft()
    rig.eng.poll()
    sc = scores[0].cpu().numpy()
    assert (np.diff(sc) <= 0).all()
    for i in (0, BW - 1):
        ref = ora.sequence_logprob(rig.D, rig.W["tok_emb"], g, h, beams[0, i].cpu().numpy(), rig.odt)
        assert abs(ref - sc[i]) < REL * abs(ref)

    # one verified step on planted beams
    rng = np.random.default_rng(41)
    planted = synth.plant_beams(cont, BW, L, cfg["vocab"], rng, p=0.3, rho=0.3)
    ref = ora.spec_step(rig.W, rig.D, cfg, kv, ctx, g, h, BW, L, planted=planted, run_drafter=False, dtype=rig.odt)
    beams_d = dev(planted[None])
    pk = rig.eng.pack(beams_d)
    argmax, hidden, logits = rig.eng.verify(pk, want_logits=True)
    out = rig.eng.accept(beams_d, pk, argmax, hidden)
    rig.eng.poll()
    n = ref["packed"]["n"]
    assert int(pk.n[0]) == n
    assert pk.tokens[0, :n].tolist() == ref["packed"]["tokens"].tolist()
    assert pk.unpack[0].cpu().numpy().tolist() == ref["packed"]["unpack"].tolist()
    assert (pk.mask_bool(0) == ref["packed"]["mask"]).all()
    assert rel_err(logits[0, :n].cpu().numpy(), ref["logits"]) < REL
    assert rel_err(hidden[0, :n].cpu().numpy(), ref["hidden"]) < REL
    am = argmax[0, :n].cpu().numpy()
    sure = decided(ref["logits"])
    assert (am[sure] == ref["argmax"][sure]).all()
    a, best, toks = ora.accept_greedy(planted, ref["packed"]["unpack"], am)
    assert int(out.n_accept[0]) == a and int(out.best[0]) == best
    assert out.tokens[0, :a + 1].tolist() == toks and (out.tokens[0, a + 1:] == -1).all()
    c_ctx, c_root, c_h = rig.eng.get_state()
    assert int(c_ctx[0]) == ctx + 1 + a and int(c_root[0]) == toks[-1]
    if a == ref["n_accept"] and toks == ref["emitted"]:
        assert rel_err(c_h[0].cpu().numpy()[None], np.asarray(ref["h"])[None]) < REL
        kvg = rig.eng.kv_view()[:, 0, 0, :, :ref["ctx"]].float().cpu().numpy().transpose(0, 2, 1, 3)
        assert np.abs(kvg - kv.k[:, :ref["ctx"]]).max() < REL * np.abs(kv.k[:, :ref["ctx"]]).max()
    rig.eng.close()

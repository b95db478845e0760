"""Parity at the benchmark's own size: the 7B workload at its full depth (32 layers), beam width 8, beam length 5,
batch 1, in the launch configuration `bench.py` times (tensor-core projections, counter hand-off, tree attention).

The oracle (fp32 numpy on the same bf16-rounded weight values) needs about 13 GFLOP per row at this depth, so the
case keeps the prompt to 32 tokens and checks ONE step: the state after the prompt, the drafter's scores for sampled
beams, packing bit-exact, the verification logits of every packed row within the bf16 bound, greedy tokens where
the oracle's gap decides them, and acceptance + hand-off bit-exact against the oracle's rule applied to the GPU's
own greedy tokens.  The beams of the verified step are planted from the GPU's own autoregressive continuation (an
input recipe, not an expected value), so that several tokens are accepted.

Tolerance.  The bf16 path stores every projection input, Q, K, V and the softmax weights that multiply V in bf16
(relative step 2^-8).  That storage is part of the path's definition, and the oracle can apply it (store="bf16":
the same arrays rounded element by element, nothing else changed); against that oracle the stated bound of 3e-2 of
the row's largest |logit| holds at the full 32 layers and is what this case asserts.  The distance to the UNROUNDED
oracle is printed, not bounded by 3e-2: the storage noise of the layers is independent and grows as the square
root of the depth, 0.7e-2 after one layer and 1.6e-2 after eight between the two oracle modes on the CPU
(tests/test_oracle_storage.py), about 3e-2 for the average row at 32 layers and more for the worst element of the
worst row.  It is only held to a loose sanity bound here.
"""
import numpy as np
import pytest
import torch

from helpers import Rig, dev, top2_gap
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu

REL = 3e-2          # against the oracle with the path's bf16 storage points
SANITY_PLAIN = 0.12  # against the unrounded oracle: reported; four times the two-mode distance the CPU test extrapolates


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
    ctx, g, h = ora.prefill(rig.W, cfg, prompt, kv, rig.odt, store="bf16")
    kv_plain = rig.new_kv()
    _, _, h_plain = ora.prefill(rig.W, cfg, prompt, kv_plain, rig.odt)
    c_ctx, c_root, c_h = rig.eng.get_state()
    rig.eng.poll()
    assert int(c_ctx[0]) == ctx == 32
    assert rel_err(c_h[0].cpu().numpy()[None], np.asarray(h)[None]) < REL
    figures = {"h after the prompt": (rel_err(c_h[0].cpu().numpy()[None], np.asarray(h)[None]),
                                      rel_err(c_h[0].cpu().numpy()[None], np.asarray(h_plain)[None]))}
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
        ref = ora.sequence_logprob(rig.D, rig.W["tok_emb"], g, h, beams[0, i].cpu().numpy(), rig.odt, store="bf16")
        assert abs(ref - sc[i]) < REL * abs(ref)

    # one verified step on planted beams
    rng = np.random.default_rng(41)
    planted = synth.plant_beams(cont, BW, L, cfg["vocab"], rng, p=0.3, rho=0.3)
    ref = ora.spec_step(rig.W, rig.D, cfg, kv, ctx, g, h, BW, L, planted=planted, run_drafter=False, dtype=rig.odt,
                        store="bf16")
    # the unrounded oracle on the same rows, from its own cache but the same root and hidden state: a reported figure
    ref_plain = ora.spec_step(rig.W, rig.D, cfg, kv_plain, ctx, g, h, BW, L, planted=planted, run_drafter=False,
                              dtype=rig.odt)
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
    got = logits[0, :n].cpu().numpy()
    figures["verification logits"] = (rel_err(got, ref["logits"]), rel_err(got, ref_plain["logits"]))
    figures["verification logits, relative L2 of the worst row"] = (
        float((np.linalg.norm(got - ref["logits"], axis=1) / np.linalg.norm(ref["logits"], axis=1)).max()),
        float((np.linalg.norm(got - ref_plain["logits"], axis=1) / np.linalg.norm(ref_plain["logits"], axis=1)).max()))
    for what, (r_store, r_plain) in figures.items():
        print(f"[7B, 32 layers] {what}: {r_store:.4f} of the row's max against the oracle with bf16 storage, "
              f"{r_plain:.4f} against the unrounded oracle")
    assert rel_err(got, ref["logits"]) < REL
    assert rel_err(hidden[0, :n].cpu().numpy(), ref["hidden"]) < REL
    assert rel_err(got, ref_plain["logits"]) < SANITY_PLAIN
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

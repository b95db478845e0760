"""The arm without tree attention (Figure 3(a), Figure 5): every candidate sends all of its tokens, only the root is
shared; verification, acceptance and KV compaction run on that flat layout.

Checked: the whole step under RD_FLAG_NO_TREE against the oracle's flat_beam + spec_step(tree=False), and -- the
property that makes dynamic tree attention lossless (Section 3.3) -- that a node of the packed tree and every copy of
it in the flat layout get the same logits on the GPU.
"""
import numpy as np
import pytest
import torch

from helpers import Rig, dev, top2_gap
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import binding, synth

pytestmark = pytest.mark.gpu

RAGGED = dict(synth.CONFIGS["tiny"], dtype="bf16", d_model=512, n_heads=4, d_ffn=1376, vocab=1000, d_rnn=512,
              max_ctx=400, beam_width=8, beam_length=5, prompt_len=96)


def rel_err(got, ref):
    return float((np.abs(got - ref) / np.abs(ref).max(axis=-1, keepdims=True)).max())


def flat_against_oracle_and_packed(cfg, tol_abs, tol_rel, n_steps, seed):
    flat = Rig(cfg=cfg, flags=binding.RD_FLAG_NO_TREE)
    tree = Rig(cfg=cfg)
    BW, L, V = cfg["beam_width"], cfg["beam_length"], cfg["vocab"]
    prompt = np.random.default_rng(seed).integers(0, V, size=cfg["prompt_len"])
    kv = flat.new_kv()
    ctx, g, h = ora.prefill(flat.W, cfg, prompt, kv)
    ar, _, _ = ora.generate_ar(flat.W, cfg, prompt, 2 + n_steps * (L + 1), cfg["max_ctx"])
    flat.eng.prefill([prompt])
    tree.eng.prefill([prompt])
    rng = np.random.default_rng(seed + 1)
    emitted, compared = [g], 0
    for step in range(n_steps):
        planted = synth.plant_beams(ar[len(emitted):len(emitted) + L], BW, L, V, rng, p=0.3, rho=0.3)
        ref = ora.spec_step(flat.W, flat.D, cfg, kv, ctx, g, h, BW, L, planted=planted, tree=False, run_drafter=False)
        h32 = dev(np.asarray(h, dtype=np.float32)[None], torch.float32)
        for r in (flat, tree):
            r.eng.set_state(dev([ctx]), dev([g]), h32, batch=1, ctx_bound=ctx)
        beams_d = dev(planted[None])
        # flat layout: pack, verify, accept
        pk = flat.eng.pack(beams_d)
        argmax, hidden, logits = flat.eng.verify(pk, want_logits=True)
        out = flat.eng.accept(beams_d, pk, argmax, hidden)
        flat.eng.poll()
        n = 1 + BW * L
        assert int(pk.n[0]) == n == ref["packed"]["n"]
        assert pk.tokens[0, :n].tolist() == ref["packed"]["tokens"].tolist()
        assert pk.unpack[0].cpu().numpy().tolist() == ref["packed"]["unpack"].tolist()
        assert pk.pos[0, :n].tolist() == ref["packed"]["pos"].tolist()
        assert (pk.mask_bool(0) == ref["packed"]["mask"]).all()
        got = logits[0, :n].cpu().numpy()
        if tol_abs is not None:
            assert np.abs(got - ref["logits"]).max() < tol_abs
        else:
            assert rel_err(got, ref["logits"]) < tol_rel
        # acceptance is the oracle's rule on the GPU's own greedy tokens, bit for bit
        am = argmax[0, :n].cpu().numpy()
        a, best, toks = ora.accept_greedy(planted, ref["packed"]["unpack"], am)
        assert int(out.n_accept[0]) == a and int(out.best[0]) == best
        assert out.tokens[0, :a + 1].tolist() == toks and (out.tokens[0, a + 1:] == -1).all()
        # packed tree on the GPU: a node and each of its flat copies see the same logits
        pk_t = tree.eng.pack(beams_d)
        argmax_t, hidden_t, logits_t = tree.eng.verify(pk_t, want_logits=True)
        tree.eng.accept(beams_d, pk_t, argmax_t, hidden_t)         # keeps this engine's cache in step with the other's
        tree.eng.poll()
        up_t, up_f = pk_t.unpack[0].cpu().numpy(), pk.unpack[0].cpu().numpy()
        lt = logits_t[0].cpu().numpy()
        assert int(pk_t.n[0]) < n                                  # prefixes were shared
        for i in range(BW):
            for j in range(L + 1):
                if tol_abs is not None:
                    assert np.abs(got[up_f[i, j]] - lt[up_t[i, j]]).max() < tol_abs
                else:
                    assert rel_err(got[up_f[i, j]][None], lt[up_t[i, j]][None]) < 1e-2
        # where the oracle's gaps decide every greedy token, the whole outcome and the compacted cache are the oracle's
        gap = 0.05 if tol_abs is not None else np.maximum(0.05, 2 * tol_rel * np.abs(ref["logits"]).max(axis=-1))
        if (top2_gap(ref["logits"]) > gap).all():
            assert a == ref["n_accept"] and best == ref["best"] and toks == ref["emitted"]
        if a == ref["n_accept"] and toks == ref["emitted"]:
            compared += 1
            c_ctx, c_root, c_h = flat.eng.get_state()
            assert int(c_ctx[0]) == ref["ctx"] and int(c_root[0]) == ref["g"]
            kvg = flat.eng.kv_view()[:, :, 0, :, :ref["ctx"]].float().cpu().numpy()
            scale = np.abs(kv.k[:, :ref["ctx"]]).max()
            tol = tol_abs if tol_abs is not None else tol_rel * scale
            assert np.abs(kvg[:, 0].transpose(0, 2, 1, 3) - kv.k[:, :ref["ctx"]]).max() < tol
            assert np.abs(kvg[:, 1].transpose(0, 2, 1, 3) - kv.v[:, :ref["ctx"]]).max() < tol
        else:
            break
        ctx, g, h = ref["ctx"], ref["g"], ref["h"]
        emitted.extend(ref["emitted"])
    flat.eng.close()
    tree.eng.close()
    return compared


def test_flat_layout_whole_step_fp32():
    assert flat_against_oracle_and_packed(dict(synth.CONFIGS["tiny"]), 2e-3, None, n_steps=6, seed=31) >= 4


def test_flat_layout_whole_step_bf16():
    assert flat_against_oracle_and_packed(dict(RAGGED), None, 3e-2, n_steps=4, seed=32) >= 2

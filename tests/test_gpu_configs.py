"""Parity at the per-layer shapes of the larger workloads (13B, 7B batch 16, 33B), depth-reduced.

With hundred-token prompts and every sequence followed, the oracle cannot run these models at full depth in
test time (tens of TFLOP per step on host cores), so each case keeps the workload's exact per-layer shapes, beam width, beam length and batch, cuts the
depth to two layers and the prompts to about a hundred tokens, and checks one planted-beam step:
packing bit-exact, verification logits within the bf16 bound, greedy tokens where the oracle's gap
decides them, acceptance + hand-off bit-exact against the oracle's rule on the GPU's own greedy tokens.

The `*_full_depth` cases run the same step at the workloads' own depth (40, 32 and 60 layers) with prompts of a few
dozen tokens, the oracle following one or two of the sequences.  Every case runs the oracle in both of its modes
(unrounded, and with the path's bf16 storage points: projection inputs, Q, K, V and the softmax weights rounded
element by element).  Every case bounds the GPU's distance to the unrounded oracle by 1.15 x the distance between the
two oracle modes of that same case -- the storage noise, which involves no kernel -- and its distance to the rounded
oracle by 1.3 x it (helpers.check_against_storage_noise).  The two-layer cases also meet the stated 3e-2
against both oracles; at full depth the storage noise alone exceeds it (3.9e-2 relative L2 at 32 layers, 5.7e-2 at 40,
8.8e-2 at 60), so no implementation that stores these arrays in bf16 can.
"""
import numpy as np
import pytest
import torch

from helpers import Rig, check_against_storage_noise, dev, top2_gap
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu

REL = 3e-2


def rel_err(got, ref):
    return float((np.abs(got - ref) / np.abs(ref).max(axis=-1, keepdims=True)).max())


def decided(ref_logits, rel=REL):
    bound = rel * np.abs(ref_logits).max(axis=-1)
    return top2_gap(ref_logits) > np.maximum(0.05, 2 * bound)


def one_step(name, prompt_lens, check_seqs, rho, layers=2):
    """layers=None: the workload's own depth."""
    base = synth.CONFIGS[name]
    B = len(prompt_lens)
    cfg = dict(base, max_batch=B, max_ctx=max(prompt_lens) + 2 + base["beam_width"] * base["beam_length"] + 8)
    if layers is not None:
        cfg = synth.with_layers(cfg, layers)
    full = layers is None
    tag = f"[{name}, {cfg['n_layers']} layers]"
    stated = None if full else REL      # the stated 3e-2 applies where the storage noise leaves room for it
    rig = Rig(cfg=cfg, oracle_dtype=np.float32)
    BW, L, V = cfg["beam_width"], cfg["beam_length"], cfg["vocab"]
    rng = np.random.default_rng(cfg["seed"])
    prompts = [rng.integers(0, V, size=n) for n in prompt_lens]
    rig.eng.prefill(prompts)
    c_ctx, c_root, c_h = rig.eng.get_state()
    rig.eng.poll()
    roots = c_root.cpu().numpy().copy()
    hs = c_h.cpu().numpy().copy()
    # planted beams around an arbitrary continuation (random tokens): shared prefixes stress the packing
    beams = np.stack([synth.plant_beams(rng.integers(0, V, size=L), BW, L, V, rng, p=0.3, rho=rho) for _ in range(B)])
    refs = {}
    for b in check_seqs:
        kv = rig.new_kv()
        ctx, g, h = ora.prefill(rig.W, cfg, prompts[b], kv, np.float32, store="bf16")
        kv_plain = rig.new_kv()
        _, _, h_plain = ora.prefill(rig.W, cfg, prompts[b], kv_plain, np.float32)
        assert int(c_ctx[b]) == ctx
        check_against_storage_noise(hs[b][None], np.asarray(h)[None], np.asarray(h_plain)[None],
                                    f"{tag} sequence {b}, h after the prompt", stated, l2_factor=1.25)   # a single row
        roots[b] = g                                    # teacher-force the oracle's root and hidden state
        hs[b] = h
        refs[b] = (kv, ctx, g, h, kv_plain)
    rig.eng.set_state(None, dev(roots), dev(hs.astype(np.float32), torch.float32))
    beams_d = dev(beams)
    pk = rig.eng.pack(beams_d)
    argmax, hidden, logits = rig.eng.verify(pk, want_logits=True)
    out = rig.eng.accept(beams_d, pk, argmax, hidden)
    rig.eng.poll()
    n_ctx, n_root, n_h = rig.eng.get_state()
    for b, (kv, ctx, g, h, kv_plain) in refs.items():
        aug = np.concatenate([np.full((BW, 1), g), beams[b]], axis=1)
        p = ora.pack_beam(aug, ctx)
        n = p["n"]
        assert int(pk.n[b]) == n
        assert pk.tokens[b, :n].tolist() == p["tokens"].tolist()
        assert pk.unpack[b].cpu().numpy().tolist() == p["unpack"].tolist()
        assert pk.pos[b, :n].tolist() == p["pos"].tolist()
        assert (pk.mask_bool(b) == p["mask"]).all()
        rh, rl = ora.llm_forward(rig.W, cfg, p["tokens"], p["pos"], p["mask"], kv, ctx, np.float32, store="bf16")
        rh_plain, rl_plain = ora.llm_forward(rig.W, cfg, p["tokens"], p["pos"], p["mask"], kv_plain, ctx, np.float32)
        got = logits[b, :n].cpu().numpy()
        check_against_storage_noise(got, rl, rl_plain, f"{tag} sequence {b}, verification logits", stated)
        check_against_storage_noise(hidden[b, :n].cpu().numpy(), rh, rh_plain, f"{tag} sequence {b}, hidden states", stated)
        am = argmax[b, :n].cpu().numpy()
        sure = decided(rl, 2 * REL if full else REL)
        assert (am[sure] == rl.argmax(1)[sure]).all()
        a, best, toks = ora.accept_greedy(beams[b], p["unpack"], am)
        assert int(out.n_accept[b]) == a and int(out.best[b]) == best
        assert out.tokens[b, :a + 1].tolist() == toks
        assert int(n_ctx[b]) == ctx + 1 + a and int(n_root[b]) == toks[-1]
        node = int(p["unpack"][best, a])
        assert np.allclose(n_h[b].cpu().numpy(), hidden[b, node].cpu().numpy())
    rows = int(pk.n.sum())
    rig.eng.close()
    return rows


def test_13b_shapes_beam_width_64():
    rows = one_step("13b", [96], [0], rho=0.5)
    assert 64 < rows <= 321                              # two activation tiles per weight tile


def test_7b_batch_16_ragged():
    lens = [int(x) for x in np.random.default_rng(4).integers(40, 121, size=16)]
    rows = one_step("7b_bs16", lens, [0, 7, 15], rho=0.3)
    assert rows > 256


def test_33b_shapes_batch_4():
    rows = one_step("33b", [64, 80, 72, 90], [1, 3], rho=0.3)
    assert rows > 128


# ---- the same step at the workloads' own depth (short prompts, the oracle follows one or two sequences)
def test_13b_full_depth():
    rows = one_step("13b", [24], [0], rho=0.5, layers=None)
    assert 64 < rows <= 321


def test_7b_batch_16_full_depth():
    lens = [int(x) for x in np.random.default_rng(5).integers(16, 41, size=16)]
    rows = one_step("7b_bs16", lens, [0, 9], rho=0.3, layers=None)
    assert rows > 256


def test_33b_full_depth():
    """60 layers: the fp32 copy of the weights for the oracle takes 133 GB of host memory, so the case runs only where
    that leaves room (it follows one of the four sequences)."""
    import psutil
    if psutil.virtual_memory().available < 170 * 2 ** 30:
        pytest.skip("needs 170 GB of free host memory for the oracle's fp32 weights")
    rows = one_step("33b", [16, 24, 20, 28], [2], rho=0.3, layers=None)
    assert rows > 128

"""Verification passes at the larger workloads' own context lengths, through the attention kernel each of them takes by
default (Section 3.4: attention over the KV cache plus the tree mask).

The library picks among four bf16 attention kernels by row count, context length and the number of (head, sequence,
row tile) CTAs.  The depth-reduced shape cases use prompts of about a hundred tokens and so never reach the kernels
that the 13B (1024-token prompt, 321 rows), the batched 7B (contexts 256-2048, batch 16) and the 33B workload
(4096-token prompts, batch 4) run on.  Each case here keeps what decides the routing -- head dimension, rows per
sequence, context length, enough CTAs -- on a model small enough for the oracle (2 layers, d_model 512-2048), runs one
planted-beam verification pass on top of a GPU-prefilled cache, checks it against the oracle element by element, and
asserts through redrafter_route_counts that the intended kernel did the work.
"""
import numpy as np
import pytest
import torch

from helpers import Rig, check_against_storage_noise, dev, top2_gap
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu

REL = 3e-2
BASE = dict(synth.CONFIGS["tiny"], dtype="bf16", n_layers=2, d_ffn=1376, vocab=1000, beam_length=5)


def decided(ref_logits):
    bound = REL * np.abs(ref_logits).max(axis=-1)
    return top2_gap(ref_logits) > np.maximum(0.05, 2 * bound)


def verify_on_long_contexts(cfg, prompt_lens, follow, rho, seed, p_replace=0.3):
    """Prefill on the GPU, then one verification pass on planted beams; the oracle follows the sequences in `follow`
    (its own prefill, both storage modes) and every one of their packed rows is compared.  Returns the route counters
    of the verification pass alone."""
    rig = Rig(cfg=cfg, oracle_dtype=np.float32)
    B, BW, L, V = len(prompt_lens), cfg["beam_width"], cfg["beam_length"], cfg["vocab"]
    rng = np.random.default_rng(seed)
    prompts = [rng.integers(0, V, size=n) for n in prompt_lens]
    rig.eng.prefill(prompts)
    c_ctx, c_root, c_h = rig.eng.get_state()
    rig.eng.poll()
    roots, hs = c_root.cpu().numpy().copy(), c_h.cpu().numpy().copy()
    beams = np.stack([synth.plant_beams(rng.integers(0, V, size=L), BW, L, V, rng, p=p_replace, rho=rho) for _ in range(B)])
    refs = {}
    for b in follow:
        kv, kv_plain = rig.new_kv(), rig.new_kv()
        ctx, g, h = ora.prefill(rig.W, cfg, prompts[b], kv, np.float32, store="bf16")
        _, _, h_plain = ora.prefill(rig.W, cfg, prompts[b], kv_plain, np.float32)
        assert int(c_ctx[b]) == ctx == prompt_lens[b]
        check_against_storage_noise(hs[b][None], np.asarray(h)[None], np.asarray(h_plain)[None],
                                    f"sequence {b} ({ctx} tokens), h after the prompt", REL, l2_factor=1.25)
        roots[b], hs[b] = g, h
        refs[b] = (kv, kv_plain, ctx, g)
    rig.eng.set_state(None, dev(roots), dev(hs.astype(np.float32), torch.float32))
    before = rig.eng.route_counts()
    beams_d = dev(beams)
    pk = rig.eng.pack(beams_d)
    argmax, hidden, logits = rig.eng.verify(pk, want_logits=True)
    rig.eng.poll()
    after = rig.eng.route_counts()
    for b, (kv, kv_plain, ctx, g) in refs.items():
        aug = np.concatenate([np.full((BW, 1), g), beams[b]], axis=1)
        p = ora.pack_beam(aug, ctx)
        n = p["n"]
        assert int(pk.n[b]) == n and pk.tokens[b, :n].tolist() == p["tokens"].tolist()
        assert (pk.mask_bool(b) == p["mask"]).all()
        rh, rl = ora.llm_forward(rig.W, cfg, p["tokens"], p["pos"], p["mask"], kv, ctx, np.float32, store="bf16")
        _, rl_plain = ora.llm_forward(rig.W, cfg, p["tokens"], p["pos"], p["mask"], kv_plain, ctx, np.float32)
        got = logits[b, :n].cpu().numpy()
        check_against_storage_noise(got, rl, rl_plain, f"sequence {b} ({ctx} tokens, {n} rows), verification logits", REL)
        sure = decided(rl)
        assert sure.sum() >= n // 4
        assert (argmax[b, :n].cpu().numpy()[sure] == rl.argmax(1)[sure]).all()
        # the provisional K rows of this pass are in the cache at slots ctx + n
        kvg = rig.eng.kv_view()[:, 0, b, :, ctx:ctx + n].float().cpu().numpy().transpose(0, 2, 1, 3)
        assert np.abs(kvg - kv.k[:, ctx:ctx + n]).max() < REL * np.abs(kv.k[:, ctx:ctx + n]).max()
    rig.eng.close()
    return {k: after[k] - before[k] for k in after}, int(pk.n.max()), int(pk.n.sum())


def test_wide_beam_long_context_takes_the_tcgen05_kernel():
    """The 13B and 33B workloads' regime: head dimension 128, beam width 32 (up to 161 rows per sequence), more than a
    thousand tokens of context, more (head, sequence, tile) CTAs than four waves of 16-row tiles: tree-masked rows
    through 128-row tcgen05 tiles, the second tile of every sequence partly filled."""
    cfg = dict(BASE, d_model=2048, n_heads=16, d_rnn=2048, max_batch=4, beam_width=32, max_ctx=1200 + 161 + 16)
    route, n_max, n_sum = verify_on_long_contexts(cfg, [1200, 1100, 1150, 1030], follow=[0, 3], rho=0.2, seed=21, p_replace=0.6)
    assert n_max > 128
    assert route["att_rows128_tc5"] == cfg["n_layers"] and route["att_rows64"] == 0 and route["att_rows16"] == 0


def test_ragged_batch_takes_the_64_row_kernel_below_a_thousand_keys():
    """Batch 16, beam width 16 (up to 81 rows per sequence), contexts from 256 to 900 tokens (4 to 15 chunks of keys):
    tree-masked 64-row tiles, every sequence with its own context length and row count."""
    cfg = dict(BASE, d_model=512, n_heads=8, d_rnn=512, max_batch=16, beam_width=16, max_ctx=900 + 81 + 16)
    lens = [int(x) for x in np.random.default_rng(22).integers(256, 901, size=16)]
    lens[0], lens[5], lens[15] = 900, 256, 640
    route, n_max, n_sum = verify_on_long_contexts(cfg, lens, follow=[0, 5, 15], rho=0.3, seed=22)
    assert n_sum > 512
    assert route["att_rows64"] == cfg["n_layers"] and route["att_rows128_tc5"] == 0 and route["att_rows16"] == 0


def test_ragged_batch_long_contexts_take_the_tcgen05_kernel():
    """The batched 7B workload's regime: batch 16, beam width 16 (up to 81 rows per sequence), contexts from 256 to 2048
    tokens (2 to 17 chunks of 128 keys): from a thousand keys up, sequences that can fill half a 128-row tile go
    through the tcgen05 kernel (head dimension 128), every sequence with its own context length and row count, most of
    every tile unused."""
    cfg = dict(BASE, d_model=1024, n_heads=8, d_rnn=1024, max_batch=16, beam_width=16, max_ctx=2048 + 81 + 16)
    lens = [int(x) for x in np.random.default_rng(22).integers(256, 2049, size=16)]
    lens[0], lens[5], lens[15] = 2048, 256, 1400
    route, n_max, n_sum = verify_on_long_contexts(cfg, lens, follow=[0, 5, 15], rho=0.3, seed=22)
    assert n_sum > 512
    assert route["att_rows128_tc5"] == cfg["n_layers"] and route["att_rows64"] == 0 and route["att_rows16"] == 0


def test_long_context_few_heads_splits_the_keys():
    """The 33B workload's context length on few CTAs: 4096-token prompts, batch 2, 4 heads, beam width 8 (41 rows):
    16-row tiles whose keys are split over several CTAs and merged by the last one to arrive."""
    cfg = dict(BASE, d_model=512, n_heads=4, d_rnn=512, max_batch=2, beam_width=8, max_ctx=4096 + 41 + 16)
    route, n_max, n_sum = verify_on_long_contexts(cfg, [4096, 3000], follow=[0], rho=0.3, seed=23)
    assert route["att_rows16"] == cfg["n_layers"] and route["att_key_split"] == cfg["n_layers"]

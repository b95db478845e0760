"""Parity at the benchmark's own size: the 7B workload at its full depth (32 layers), beam width 8, beam length 5,
batch 1, in the launch configuration `bench.py` times (tensor-core projections, counter hand-off, tree attention).

The oracle (fp32 numpy on the same bf16-rounded weight values) needs about 13 GFLOP per row at this depth, so the
case keeps the prompt to 32 tokens and checks ONE step: the state after the prompt, the drafter's scores for sampled
beams, packing bit-exact, the verification logits of every packed row within the bf16 bound, greedy tokens where
the oracle's gap decides them, and acceptance + hand-off bit-exact against the oracle's rule applied to the GPU's
own greedy tokens.  The beams of the verified step are planted from the GPU's own autoregressive continuation (an
input recipe, not an expected value), so that several tokens are accepted.

Tolerance.  The bf16 path stores every projection input, Q, K, V and the softmax weights that multiply V in bf16
(relative step 2^-8).  The oracle can apply the same storage (store="bf16": those arrays rounded element by element,
nothing else changed).  Between the oracle's two modes -- no kernel involved -- the logits differ by 0.7e-2 (relative
L2) after one layer of this shape and 1.6e-2 after eight, growing as the square root of the depth
(tests/test_oracle_storage.py), and by 3.9e-2 at the 32 layers of this case (worst element 4.8e-2 of the row's
largest logit): the stated 3e-2 cannot be met at this depth by ANY implementation that stores these arrays in bf16,
the rounded oracle included.  Nor can an implementation be held to a tight bound against the rounded oracle: a
difference in the last bits of an fp32 sum flips bf16 roundings downstream, and two correct implementations drift
apart by 0.5 to 1 times the storage noise within eight layers (same test file).  So this case computes BOTH oracle
modes on its own rows and requires the GPU to lie no further from the unrounded oracle than 1.15 x the rounded
oracle does, nor further than 1.3 x that from the rounded oracle (helpers.check_against_storage_noise; measured 0.0395
against 0.0399, and 0.0283).  The stated 3e-2 is asserted by the two-layer copies of every workload.
"""
import numpy as np
import pytest
import torch

from helpers import check_against_storage_noise, dev, first_mismatch, Rig, top2_gap
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu

REL = 3e-2          # the stated tolerance; at this depth the bound comes from the oracle pair (see the module docstring)


def rel_err(got, ref):
    return float((np.abs(got - ref) / np.abs(ref).max(axis=-1, keepdims=True)).max())


def decided(ref_logits):
    bound = 2 * REL * np.abs(ref_logits).max(axis=-1)    # twice the stated tolerance at this depth
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
    check_against_storage_noise(c_h[0].cpu().numpy()[None], np.asarray(h)[None], np.asarray(h_plain)[None],
                                "[7B, 32 layers] h after the prompt", l2_factor=1.25)   # a single row
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
    fig = check_against_storage_noise(got, ref["logits"], ref_plain["logits"], "[7B, 32 layers] verification logits")
    assert fig["ru_max"] > REL      # at this depth the storage noise alone exceeds the stated tolerance
    check_against_storage_noise(hidden[0, :n].cpu().numpy(), ref["hidden"], ref_plain["hidden"], "[7B, 32 layers] hidden states")
    am = argmax[0, :n].cpu().numpy()
    sure = decided(ref["logits"])
    assert (am[sure] == ref["argmax"][sure]).all()
    a, best, toks = ora.accept_greedy(planted, ref["packed"]["unpack"], am)
    assert int(out.n_accept[0]) == a and int(out.best[0]) == best
    assert out.tokens[0, :a + 1].tolist() == toks and (out.tokens[0, a + 1:] == -1).all()
    c_ctx, c_root, c_h = rig.eng.get_state()
    assert int(c_ctx[0]) == ctx + 1 + a and int(c_root[0]) == toks[-1]
    if a == ref["n_accept"] and toks == ref["emitted"]:
        kvg = rig.eng.kv_view()[:, 0, 0, :, :ref["ctx"]].float().cpu().numpy().transpose(0, 2, 1, 3)
        assert np.abs(kvg - kv.k[:, :ref["ctx"]]).max() < 2 * REL * np.abs(kv.k[:, :ref["ctx"]]).max()
    rig.eng.close()


def test_verification_and_autoregressive_paths_differ_by_storage_noise_only():
    """Why a speculative stream in bf16 can part from the autoregressive one ("bonus flips").

    The verification pass and the autoregressive step of this library sum in different orders (tree keys at provisional
    slots, other attention chunking, other projection row counts), so at full depth their logits for the same token
    position are two samples of the storage noise.  This case runs the 7B workload's autoregressive stream, keeps its
    logits, then verifies planted beams around that stream for 24 steps and compares, at every packed node that lies on
    the stream, the verification logits with the autoregressive logits of the same position:
      * their distance stays within 1.5 x the storage noise of this depth (the worst element between the oracle's two
        modes on one step's rows, computed here; no kernel involved in that bound) -- two samples of the same noise;
      * consequently the greedy tokens of the two paths differ only at positions whose autoregressive top-2 gap is
        below twice that bound; every such position is printed with its gap.  A flip at a larger gap fails."""
    cfg = dict(synth.CONFIGS["7b"], max_ctx=512)
    rig = Rig(cfg=cfg, oracle_dtype=np.float32)
    BW, L, V = cfg["beam_width"], cfg["beam_length"], cfg["vocab"]
    n_steps = 24
    prompt = np.random.default_rng(42).integers(0, V, size=32)
    P = len(prompt)

    # the storage noise of one step's rows at this depth, from the oracle pair alone
    kv_s, kv_p = rig.new_kv(), rig.new_kv()
    ctx, g, h = ora.prefill(rig.W, cfg, prompt, kv_s, rig.odt, store="bf16")
    ora.prefill(rig.W, cfg, prompt, kv_p, rig.odt)
    rng = np.random.default_rng(43)
    probe = synth.plant_beams(rng.integers(0, V, size=L), BW, L, V, rng, p=0.3, rho=0.3)
    aug = np.concatenate([np.full((BW, 1), g), probe], axis=1)
    p0 = ora.pack_beam(aug, ctx)
    _, z_s = ora.llm_forward(rig.W, cfg, p0["tokens"], p0["pos"], p0["mask"], kv_s, ctx, rig.odt, store="bf16")
    _, z_p = ora.llm_forward(rig.W, cfg, p0["tokens"], p0["pos"], p0["mask"], kv_p, ctx, rig.odt)
    noise = float((np.abs(z_s - z_p).max(axis=1) / np.abs(z_p).max(axis=1)).max())
    assert 0.02 < noise < 0.1

    # the autoregressive stream and its logits
    n_tok = n_steps * (L + 1) + L + 1
    rig.eng.prefill([prompt])
    tok = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    stream = [int(rig.eng.get_state()[1][0])]
    z_ar = torch.empty(n_tok, V, dtype=torch.float32, device="cuda:0")
    for i in range(n_tok):
        rig.eng.ar_step(tok)
        z_ar[i].copy_(rig.eng.last_logits(1)[0])
        stream.append(int(tok[0]))
    rig.eng.poll()
    z_ar = z_ar.cpu().numpy()          # z_ar[i] chooses stream[i + 1]
    assert (z_ar.argmax(1) == np.array(stream[1:])).all()

    # planted-beam verification along the stream, root teacher-forced to the stream's own token
    rig.eng.prefill([prompt])
    pos, worst, flips, nodes = 0, 0.0, [], 0
    for step in range(n_steps):
        planted = synth.plant_beams(stream[pos + 1:pos + 1 + L], BW, L, V, rng, p=0.3, rho=0.3)
        rig.eng.set_state(None, dev([stream[pos]]), None)
        beams_d = dev(planted[None])
        pk = rig.eng.pack(beams_d)
        argmax, hidden, logits = rig.eng.verify(pk, want_logits=True)
        out = rig.eng.accept(beams_d, pk, argmax, hidden)
        rig.eng.poll()
        match = first_mismatch(planted, stream[pos + 1:pos + 1 + L])
        best = int(match.argmax())
        up = pk.unpack[0, best].cpu().numpy()
        lg = logits[0].cpu().numpy()
        for j in range(int(match[best]) + 1):              # nodes of the tree that lie on the stream
            zs, za = lg[up[j]], z_ar[pos + j]
            scale = np.abs(za).max()
            delta = float(np.abs(zs - za).max() / scale)
            worst = max(worst, delta)
            nodes += 1
            if int(zs.argmax()) != int(za.argmax()):
                top2 = np.sort(za)[-2:]
                flips.append((step, j, float((top2[1] - top2[0]) / scale), delta))
        a = int(out.n_accept[0])
        assert a <= int(match[best])                       # accepted tokens are stream tokens
        pos += a + 1
    rig.eng.close()
    print(f"[7B, 32 layers] verification vs autoregressive logits at {nodes} stream positions: worst element {worst:.4f} of "
          f"the row's max; storage noise of this depth (oracle pair) {noise:.4f}; greedy tokens differ at {len(flips)} positions")
    for step, j, gap, delta in flips:
        print(f"    step {step} depth {j}: autoregressive top-2 gap {gap:.4f} of the row's max, path distance {delta:.4f}")
    assert nodes >= 3 * n_steps
    assert worst <= 1.5 * noise
    assert all(gap <= 2 * 1.5 * noise for _, _, gap, _ in flips)

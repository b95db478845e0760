"""The drafter's beams on the GPU against the oracle's beam search, unconditionally (Section 3.2).

Beam search "ranks by probability": the result is discrete and decided by floating-point scores.  Every case compares
the GPU's beams and scores with helpers.tolerant_beam_search -- the oracle's beam search with each top-BW decision
widened by an error bound -- through helpers.check_beams_within: every beam the bound makes certain is present, no beam
the bound rules out is, every score is its sequence's log-probability, and ranks follow the oracle's scores wherever
they are further apart than twice the bound (tests/test_beam_protocol.py shows on the CPU that this rejects a selection
that returns the (k+1)-th candidate for the k-th).  The comparison is never skipped: each case asserts how many beams
the bound left certain and how many ranks it fixed exactly, and where no decision at all was within the bound the
beams must equal the oracle's element by element.

Error bounds.  fp32 path: sums of up to 1024 products in fp32 on both sides; scores (about -25) agreed to 3e-6 on 48
state vectors; bound 2e-5.  bf16 path, against the oracle with the same bf16 storage points (store="bf16"): both round
the same arrays, a last-bit difference between two fp32 sums flips an occasional rounding; measured at most 5.7e-4 over
48 state vectors and beam widths 8, 33 and 64; bound 2e-3.  (Against the unrounded oracle the scores differ by 7e-3.)
The workloads' random-init drafter barely depends on its state (embeddings of std 0.02 next to a unit-rms h), so the
best candidates of a call lie within 0.06 of each other and sequences that permute the same tokens within 1e-3:
near-ties are inherent to this input distribution, which is why the bf16 cases fix fewer ranks exactly than they
make certain.  Larger weights do not help: the head's gain per layer passes 1 (std 0.05 and up) and the rounding
flips are amplified faster than the gaps grow (measured error 2e-3 at std 0.04, 5e-3 at 0.05, 1.3e-1 at 0.12).
"""
import numpy as np
import pytest
import torch

from helpers import Rig, check_beams_within, dev, tolerant_beam_search
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu

RAGGED = dict(synth.CONFIGS["tiny"], dtype="bf16", d_model=512, n_heads=4, d_ffn=1376, vocab=1000, d_rnn=512,
              max_ctx=400, beam_width=8, beam_length=5, prompt_len=96)
N_STATES = 6


def states(cfg, n=N_STATES):
    """Drafter inputs: a root token and a unit-rms hidden vector (what a final RMSNorm with gain 1 hands over)."""
    for seed in range(n):
        rng = np.random.default_rng(100 + seed)
        g = int(rng.integers(0, cfg["vocab"]))
        h = rng.standard_normal(cfg["d_model"])
        yield g, (h / np.sqrt((h * h).mean())).astype(np.float32)


def run_case(cfg, store, eps, std, min_sure, min_fixed, min_exact):
    rig = Rig(cfg=cfg, std=std)
    BW, L = cfg["beam_width"], cfg["beam_length"]
    n_sure = n_fixed = n_exact = 0
    for g, h in states(cfg):
        rig.eng.set_state(dev([50]), dev([g]), dev(h[None], torch.float32), batch=1, ctx_bound=50)
        beams, scores = rig.eng.draft()
        rig.eng.poll()
        bm, sc = beams[0].cpu().numpy(), scores[0].cpu().numpy()
        h64 = h.astype(np.float64)
        sets = tolerant_beam_search(ora, rig.D, rig.W["tok_emb"], g, h64, BW, L, eps, store=store)
        assert sets is not None
        fixed = check_beams_within(sets, bm, sc, eps)
        n_sure += len(sets[0])
        n_fixed += fixed
        if not sets[1] and sets[2] == 0 and fixed == BW:
            # no decision of any call came within the bound: the beams are the oracle's, element by element
            rb, rs = ora.beam_search(rig.D, rig.W["tok_emb"], g, h64, BW, L, store=store)
            assert bm.tolist() == rb.tolist()
            assert np.abs(sc - rs).max() <= eps
            n_exact += 1
    rig.eng.close()
    print(f"BW {BW} std {std} eps {eps}: {n_sure} of {N_STATES * BW} beams certain, {n_fixed} ranks fixed exactly, "
          f"{n_exact} of {N_STATES} beam sets equal to the oracle's element by element")
    # the comparison took place: these counts are the oracle's (they do not depend on the GPU)
    assert n_sure >= min_sure and n_fixed >= min_fixed and n_exact >= min_exact, (n_sure, n_fixed, n_exact)


def test_fp32_beam_width_4():
    cfg = dict(synth.CONFIGS["tiny"])
    run_case(cfg, None, 2e-5, 0.02, min_sure=24, min_fixed=24, min_exact=6)


def test_fp32_beam_width_16():
    cfg = dict(synth.CONFIGS["tiny"], beam_width=16, max_ctx=64 + 2 + 16 * 4 + 8)
    run_case(cfg, None, 2e-5, 0.02, min_sure=96, min_fixed=86, min_exact=3)


@pytest.mark.parametrize("bw,min_sure,min_fixed", [(8, 36, 8), (33, 155, 14), (64, 320, 18)])
def test_bf16_two_kernel_selection(bw, min_sure, min_fixed):
    """Beam widths 8, 33 and 64 go through the segment + merge selection kernels (above 16 with sorted segment keys and
    register-resident merge candidates)."""
    cfg = dict(RAGGED, beam_width=bw, max_ctx=96 + 2 + bw * 5 + 8)
    run_case(cfg, "bf16", 2e-3, 0.02, min_sure, min_fixed, min_exact=0)

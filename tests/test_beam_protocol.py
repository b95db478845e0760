"""The comparison protocol for drafter beams (helpers.tolerant_beam_search / check_beams_within), on the CPU.

Beam search ranks candidates by floating-point scores (Section 3.2), so two correct implementations may differ where
scores are closer than their error.  The protocol widens every top-BW decision of the oracle by an error bound and
fixes everything else exactly.  These cases show that it accepts the oracle's own result and rejects the mistakes a
selection kernel can make: the (k+1)-th best candidate returned for the k-th, two ranks swapped, a score that is not
the sequence's log-probability, a repeated sequence.
"""
import numpy as np
import pytest

from helpers import check_beams_within, tolerant_beam_search
from oracle import redrafter_oracle as ora
from paper_2403_09919_b200 import synth

CFG = dict(synth.CONFIGS["tiny"], d_model=64, n_heads=2, d_ffn=128, vocab=200, d_rnn=64, n_layers=1)
BW, L, EPS = 6, 4, 1e-3


@pytest.fixture(scope="module")
def case():
    W, D = synth.weights_to_numpy(synth.make_weights(CFG, "cpu", std=0.3), CFG)
    W, D = ora.convert_weights(W, D, np.float64)
    rng = np.random.default_rng(0)
    h = rng.standard_normal(CFG["d_model"])
    g = 7
    sets = tolerant_beam_search(ora, D, W["tok_emb"], g, h, BW, L, EPS)
    beams, scores, cand = ora.beam_search(D, W["tok_emb"], g, h, BW, L, return_logp=True)
    parents, _ = ora.beam_search(D, W["tok_emb"], g, h, BW, L - 1)
    return sets, beams, scores, cand[-1], parents


def test_the_oracles_own_beams_pass_and_are_fixed_exactly(case):
    sets, beams, scores, _, _ = case
    sure, maybe, widened = sets
    assert len(sure) == BW and not maybe and widened == 0        # decisions clear of the bound by construction
    assert check_beams_within(sets, beams, scores, EPS) == BW
    # a larger bound widens the decisions instead of failing
    loose = tolerant_beam_search(ora, *_args(case), 0.5)
    assert len(loose[1]) > 0 and check_beams_within(loose, beams, scores, 0.5) < BW


def _args(case):
    W, D = synth.weights_to_numpy(synth.make_weights(CFG, "cpu", std=0.3), CFG)
    W, D = ora.convert_weights(W, D, np.float64)
    return D, W["tok_emb"], 7, np.random.default_rng(0).standard_normal(CFG["d_model"]), BW, L


def test_next_best_candidate_in_place_of_any_rank_is_rejected(case):
    sets, beams, scores, last, parents = case
    V = CFG["vocab"]
    order = np.lexsort((np.arange(last.shape[0]), -last))
    c = int(order[BW])                                            # the (BW+1)-th best candidate of the last call
    intruder = list(parents[c // V]) + [c % V]
    for k in range(BW):
        b, s = beams.copy(), scores.copy()
        b[k:-1], s[k:-1] = beams[k + 1:], scores[k + 1:]         # rank k dropped, the rest moves up
        b[-1], s[-1] = intruder, last[c]
        with pytest.raises(AssertionError):
            check_beams_within(sets, b, s, EPS)


def test_swapped_ranks_wrong_score_and_duplicates_are_rejected(case):
    sets, beams, scores, _, _ = case
    b, s = beams.copy(), scores.copy()
    b[[1, 2]] = b[[2, 1]]                                         # sequences swapped under sorted scores
    with pytest.raises(AssertionError):
        check_beams_within(sets, b, s, EPS)
    b, s = beams.copy(), scores.copy()
    s[3] += 5 * EPS
    s = np.sort(s)[::-1]
    with pytest.raises(AssertionError):
        check_beams_within(sets, b, s, EPS)
    b, s = beams.copy(), scores.copy()
    b[4] = b[3]
    with pytest.raises(AssertionError):
        check_beams_within(sets, b, s, EPS)


def test_near_ties_are_left_open_but_nothing_else():
    """Two candidates made equal on purpose (the same token twice in the vocabulary): either may be returned, every
    other rank is still fixed."""
    W, D = synth.weights_to_numpy(synth.make_weights(CFG, "cpu", std=0.3), CFG)
    W, D = ora.convert_weights(W, D, np.float64)
    h = np.random.default_rng(0).standard_normal(CFG["d_model"])
    b0, _ = ora.beam_search(D, W["tok_emb"], 7, h, BW, 1)
    twin = int(b0[BW - 1, 0])                                      # the BW-th best first token ...
    other = (twin + 1) % CFG["vocab"]
    D["draft_out"][other] = D["draft_out"][twin]                   # ... now has an exact twin: a tie at the boundary
    W["tok_emb"][other] = W["tok_emb"][twin]
    sets = tolerant_beam_search(ora, D, W["tok_emb"], 7, h, BW, 1, EPS)
    sure, maybe, widened = sets
    assert len(sure) == BW - 1 and set(maybe) == {(twin,), (other,)} and widened == 1
    beams, scores = ora.beam_search(D, W["tok_emb"], 7, h, BW, 1)
    assert check_beams_within(sets, beams, scores, EPS) == BW - 1
    alt = beams.copy()
    alt[BW - 1, 0] = other if beams[BW - 1, 0] == twin else twin
    assert check_beams_within(sets, alt, scores, EPS) == BW - 1

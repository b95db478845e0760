"""Pins of the oracle's token choice at temperature > 0 (Section 3.4: acceptance by rejection sampling).

What fixes it: the generator's published known answers, the Gumbel distribution's moments, sample frequencies
against the softmax, the accept/resample rule of speculative sampling worked out exactly for point-mass proposals,
and the property the paper states for the whole method: the generated sequence is the LLM's own.
"""
from fractions import Fraction

import numpy as np

from helpers import MICRO, micro_model, read_golden
from oracle import redrafter_oracle as ora


def test_philox_known_answers():
    rows = read_golden("philox4x32_10_known_answers.txt")
    assert len(rows) == 3
    for ln in rows:
        c, k, o = [[int(x, 16) for x in part.split()] for part in ln.split("|")]
        got = [int(x) for x in ora.philox4x32(c, k)]
        assert got == o
    # vectorised call == scalar calls, every word of the counter and of the key matters
    base = [int(x) for x in ora.philox4x32((5, 6, 7, 8), (9, 10))]
    vec = ora.philox4x32((np.arange(4, 8), 6, 7, 8), (9, 10))
    assert [int(w[1]) for w in vec] == base
    for i in range(4):
        c = [5, 6, 7, 8]
        c[i] += 1
        assert [int(x) for x in ora.philox4x32(c, (9, 10))] != base
    assert [int(x) for x in ora.philox4x32((5, 6, 7, 8), (9, 11))] != base
    assert [int(x) for x in ora.philox4x32((5, 6, 7, 8), (10, 10))] != base


def test_uniform_is_open_and_exact_in_fp32():
    u = ora.uniform_open(np.array([0, 0x1FF, 0x200, 0xFFFFFFFF], dtype=np.uint64))
    assert u.tolist() == [2.0 ** -24, 2.0 ** -24, 3 * 2.0 ** -24, 1 - 2.0 ** -24]
    assert (u.astype(np.float32).astype(np.float64) == u).all()


def test_gumbel_moments_and_keying():
    g = ora.gumbel_noise(seed=11, seq=0, pos=3, vocab=200001)
    assert g.shape == (200001,)
    assert abs(g.mean() - 0.5772156649) < 0.01            # Euler-Mascheroni
    assert abs(g.var() - np.pi ** 2 / 6) < 0.03
    assert abs(np.median(g) + np.log(np.log(2.0))) < 0.01
    # a prefix of a longer vocabulary is the same noise; (seed, seq, pos) each select another stream
    assert (ora.gumbel_noise(11, 0, 3, 10) == g[:10]).all()
    for other in (ora.gumbel_noise(12, 0, 3, 10), ora.gumbel_noise(11, 1, 3, 10), ora.gumbel_noise(11, 0, 4, 10),
                  ora.gumbel_noise(11 + (1 << 32), 0, 3, 10)):
        assert not np.allclose(other, g[:10])
    a, b = ora.gumbel_noise(11, 0, 4, 200000), ora.gumbel_noise(11, 0, 5, 200000)
    assert abs(np.corrcoef(a, b)[0, 1]) < 0.01
    assert abs(np.corrcoef(a[:-1], a[1:])[0, 1]) < 0.01


def softmax(z):
    e = np.exp(z - z.max())
    return e / e.sum()


def test_frequencies_follow_the_softmax():
    logits = np.array([1.0, -0.5, 0.3, 2.0, 0.0, -3.0])            # ragged against the generator's four words
    for T in (0.7, 1.0, 2.5):
        smp = dict(temperature=T, seed=1234)
        n = 40000
        counts = np.bincount([ora.choose_token(logits, smp, seq=2, pos=p) for p in range(n)], minlength=6)
        expect = softmax(logits / T) * n
        chi2 = ((counts - expect) ** 2 / expect).sum()
        assert chi2 < 25.7, (T, chi2)                                # 5 degrees of freedom, p = 1e-4


def test_low_temperature_and_none_are_greedy():
    rng = np.random.default_rng(0)
    for _ in range(20):
        z = rng.normal(size=50)
        assert ora.choose_token(z, None) == int(np.argmax(z))
        assert ora.choose_token(z, dict(temperature=0.0, seed=5)) == int(np.argmax(z))
        gap = np.sort(z)[-1] - np.sort(z)[-2]
        if gap > 1e-2:
            assert ora.choose_token(z, dict(temperature=1e-4, seed=5), pos=7) == int(np.argmax(z))


def textbook_law(p, children):
    """Output law of speculative sampling's accept/resample rule when the proposals are the given tokens, tried in
    order, each a point mass (q = 1 on the proposed token): returns (P[descend to child c] for each c,
    law of the token emitted when every child was rejected), in exact arithmetic."""
    p = [Fraction(x) for x in p]
    descend, alive = [], Fraction(1)
    for c in children:
        q = [Fraction(int(v == c)) for v in range(len(p))]
        acc = min(Fraction(1), p[c] / q[c])
        descend.append(alive * acc)
        alive *= 1 - acc
        if alive == 0:
            break
        resid = [max(Fraction(0), p[v] - q[v]) for v in range(len(p))]
        p = [r / sum(resid) for r in resid]
    return descend, alive, p


def test_accept_resample_rule_equals_one_draw_from_p():
    # exact: with point-mass proposals the rule descends to child c with probability p(c) and otherwise emits a
    # token distributed as p restricted to the non-children -- i.e. the law of "draw y ~ p, descend iff y is a child"
    p = [Fraction(1, 10), Fraction(3, 10), Fraction(1, 20), Fraction(1, 4), Fraction(3, 10)]
    for children in ([1], [3, 0], [4, 1, 2], [0, 1, 2, 3]):
        descend, rejected_all, law = textbook_law(p, children)
        for c, pc in zip(children, descend):
            assert pc == p[c]
        rest = 1 - sum(p[c] for c in children)
        assert rejected_all == rest
        for v in range(len(p)):
            assert law[v] == (0 if v in children else p[v] / rest)
    # the oracle's realisation: frequencies of "the draw equals the child"
    logits = np.log(np.array([float(x) for x in p]))
    smp = dict(temperature=1.0, seed=99)
    n = 30000
    draws = np.array([ora.choose_token(logits, smp, seq=0, pos=t) for t in range(n)])
    for c in range(5):
        f = (draws == c).mean()
        assert abs(f - float(p[c])) < 4 * np.sqrt(float(p[c]) * (1 - float(p[c])) / n)


def test_speculative_equals_plain_sampled_decoding():
    cfg, W, D, _ = micro_model()
    rng = np.random.default_rng(1)
    bw, L = cfg["beam_width"], cfg["beam_length"]
    total_accepted = 0
    for T, seed in ((0.3, 1), (1.0, 2), (1.0, 1 << 40)):
        smp = dict(temperature=T, seed=seed)
        prompt = rng.integers(0, cfg["vocab"], size=cfg["prompt_len"])
        spec, acc, _, ctx = ora.generate_spec(W, D, cfg, prompt, 6, bw, L, cfg["max_ctx"], sampling=smp, seq=3)
        plain, _, _ = ora.generate_ar(W, cfg, prompt, len(spec), cfg["max_ctx"], sampling=smp, seq=3)
        assert spec == plain
        assert ctx == cfg["prompt_len"] + len(spec) - 1
        total_accepted += sum(acc)
        greedy, _, _ = ora.generate_ar(W, cfg, prompt, len(spec), cfg["max_ctx"])
        if T >= 1.0:
            assert plain != greedy                         # the draws do move the sequence
        other, _, _ = ora.generate_ar(W, cfg, prompt, len(spec), cfg["max_ctx"], sampling=smp, seq=4)
        assert other != plain                              # and sequences draw independently
    # planted beams that continue the sampled sequence are accepted whole, whatever else is in the beam
    smp = dict(temperature=1.0, seed=7)
    prompt = rng.integers(0, cfg["vocab"], size=cfg["prompt_len"])
    plain, _, _ = ora.generate_ar(W, cfg, prompt, 1 + 3 * (L + 1), cfg["max_ctx"], sampling=smp)

    def planted(step, n_out, g):
        beams = rng.integers(0, cfg["vocab"], size=(bw, L))
        beams[bw - 1] = plain[n_out:n_out + L]
        return beams

    spec, acc, _, _ = ora.generate_spec(W, D, cfg, prompt, 3, bw, L, cfg["max_ctx"], planted_fn=planted, sampling=smp)
    assert acc == [L, L, L] and spec == plain

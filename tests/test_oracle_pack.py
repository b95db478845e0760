"""Pins for the oracle's dedup_prefix / pack_beam / accept (Section 3.3, Appendix A.1, Section 3.4)."""
import itertools

import numpy as np

from helpers import first_mismatch, read_golden
from oracle import redrafter_oracle as ora


def _golden_example():
    lines = read_golden("dedup_prefix_example.txt")
    b0 = lines.index("beam")
    p0 = lines.index("prefix_tree")
    beam = np.array([[int(t) for t in ln.split()] for ln in lines[b0 + 1:p0]])
    tree = np.array([[int(t) for t in ln.split()] for ln in lines[p0 + 1:]])
    return beam, tree


def test_dedup_matches_printed_example():
    beam, tree = _golden_example()
    got = ora.dedup_prefix(beam)
    assert got.tolist() == tree.tolist()
    assert got[2][1] == 0                      # the appendix's prose reading


def _first_owner_by_dict(beam):
    """Independent formulation: walk the candidates in order and remember, in a
    dictionary keyed by the prefix tuple, who showed each prefix first."""
    first = {}
    out = np.zeros(beam.shape, dtype=np.int64)
    for i, row in enumerate(beam):
        for j in range(len(row)):
            out[i, j] = first.setdefault(tuple(row[:j + 1]), i)
    return out


def test_dedup_exhaustive_small():
    for bw, bl, v in ((3, 3, 3), (4, 2, 3), (2, 4, 2)):
        for flat in itertools.product(range(v), repeat=bw * bl):
            beam = np.array(flat).reshape(bw, bl)
            assert ora.dedup_prefix(beam).tolist() == _first_owner_by_dict(beam).tolist()


def test_dedup_identical_and_distinct_rows():
    same = np.tile(np.array([[5, 6, 7]]), (4, 1))
    assert ora.dedup_prefix(same).tolist() == [[0, 0, 0]] * 4
    distinct = np.array([[1, 9, 9], [2, 9, 9], [3, 9, 9]])
    assert ora.dedup_prefix(distinct).tolist() == [[0, 0, 0], [1, 1, 1], [2, 2, 2]]


def test_pack_fig3_counts():
    g = {k: int(v) for k, v in (ln.split() for ln in read_golden("fig3_counts.txt"))}
    # Three candidates of five tokens; candidates 2 and 3 share a three-token prefix and
    # the flattened 15 tokens shrink to 8: candidate 1 must then share four tokens with one of them.
    beams = np.array([[10, 11, 12, 13, 14],
                      [10, 11, 12, 13, 15],
                      [10, 11, 12, 16, 17]])
    assert beams.size == g["flattened"]
    aug = np.concatenate([np.full((3, 1), 99), beams], axis=1)
    p = ora.pack_beam(aug, ctx=0)
    assert p["n"] - 1 == g["deduplicated"]          # root excluded
    assert (beams[1, :3] == beams[2, :3]).all() and beams[1, 3] != beams[2, 3]


def test_pack_worked_example_with_root():
    beam, _ = _golden_example()
    g = 7
    aug = np.concatenate([np.full((3, 1), g), beam], axis=1)
    p = ora.pack_beam(aug, ctx=100)
    assert p["tokens"].tolist() == [g, 91, 92, 93, 95, 94, 96, 97]
    assert p["unpack"].tolist() == [[0, 1, 2, 3, 4], [0, 1, 2, 5, 6], [0, 1, 2, 3, 7]]
    assert p["depth"].tolist() == [0, 1, 2, 3, 4, 3, 4, 4]
    assert p["pos"].tolist() == [100, 101, 102, 103, 104, 103, 104, 104]
    assert p["parent"].tolist() == [-1, 0, 1, 2, 3, 2, 5, 3]
    rows = [set(np.nonzero(r)[0].tolist()) for r in p["mask"]]
    assert rows == [{0}, {0, 1}, {0, 1, 2}, {0, 1, 2, 3}, {0, 1, 2, 3, 4}, {0, 1, 2, 5},
                    {0, 1, 2, 5, 6}, {0, 1, 2, 3, 7}]


def _check_pack_invariants(aug, p):
    bw, cols = aug.shape
    prefixes = {tuple(aug[i, :j + 1]) for i in range(bw) for j in range(cols)}
    assert p["n"] == len(prefixes)                                     # one node per distinct prefix
    for i in range(bw):
        for j in range(cols):
            assert p["tokens"][p["unpack"][i, j]] == aug[i, j]         # unpack o pack = identity
    n = p["n"]
    assert p["parent"][0] == -1 and (p["parent"][1:] >= 0).all()
    assert (p["parent"][1:] < np.arange(1, n)).all()                   # parents precede children
    for r in range(n):
        anc, q = set(), r
        while q >= 0:
            anc.add(q)
            q = int(p["parent"][q])
        assert set(np.nonzero(p["mask"][r])[0].tolist()) == anc        # mask = closure of parent
        assert p["mask"][r].sum() == p["depth"][r] + 1
    for i in range(bw):
        assert (np.diff(p["unpack"][i]) > 0).all()                     # path rows strictly increase


def test_pack_invariants_random():
    rng = np.random.default_rng(0)
    for trial in range(300):
        bw = int(rng.integers(1, 9))
        L = int(rng.integers(1, 6))
        v = int(rng.integers(2, 5))
        beams = rng.integers(0, v, size=(bw, L))
        aug = np.concatenate([np.full((bw, 1), 3), beams], axis=1)
        _check_pack_invariants(aug, ora.pack_beam(aug, ctx=int(rng.integers(0, 50))))


def test_pack_edge_cases():
    L = 4
    same = np.tile(np.array([[1, 2, 3, 4]]), (5, 1))
    p = ora.pack_beam(np.concatenate([np.zeros((5, 1), int), same], axis=1), 0)
    assert p["n"] == 1 + L
    distinct = np.arange(5)[:, None] * 10 + np.arange(L)[None, :]
    p = ora.pack_beam(np.concatenate([np.zeros((5, 1), int), distinct], axis=1), 0)
    assert p["n"] == 1 + 5 * L
    p = ora.pack_beam(np.array([[9, 1, 2, 3]]), 4)                      # beam width 1: a chain
    assert p["n"] == 4 and p["parent"].tolist() == [-1, 0, 1, 2]


def test_flat_beam_is_per_candidate_causal():
    rng = np.random.default_rng(1)
    beams = rng.integers(0, 3, size=(4, 3))
    aug = np.concatenate([np.full((4, 1), 2), beams], axis=1)
    p = ora.flat_beam(aug, 10)
    assert p["n"] == 1 + 4 * 3
    for i in range(4):
        for j in range(4):
            assert p["tokens"][p["unpack"][i, j]] == aug[i, j]
            assert set(np.nonzero(p["mask"][p["unpack"][i, j]])[0]) == set(p["unpack"][i, :j + 1])


def test_accept_brute_force_and_planted_closed_form():
    from paper_2403_09919_b200 import synth
    rng = np.random.default_rng(2)
    V, L = 50, 5
    for trial in range(200):
        bw = int(rng.integers(1, 9))
        cont = rng.integers(0, V, size=L + 1)          # the LLM's greedy continuation after the root
        beams = synth.plant_beams(cont, bw, L, V, rng, p=0.3, rho=0.5 if trial % 2 else 0.0)
        aug = np.concatenate([np.full((bw, 1), 1), beams], axis=1)
        p = ora.pack_beam(aug, 0)
        # an LLM that continues every on-path node with the continuation and says V (never a
        # drafted token) elsewhere
        am = np.full(p["n"], V)
        for i in range(bw):
            for j in range(L + 1):
                if (aug[i, 1:j + 1] == cont[:j]).all():
                    am[p["unpack"][i, j]] = cont[j]
        a, best, emitted = ora.accept_greedy(beams, p["unpack"], am)
        ai = first_mismatch(beams, cont)
        assert a == ai.max()
        assert best == int(np.argmax(ai))               # lowest index among the longest
        assert emitted == cont[:a + 1].tolist()


def test_accept_zero_and_full():
    beams = np.array([[5, 6], [7, 8]])
    aug = np.concatenate([np.full((2, 1), 1), beams], axis=1)
    p = ora.pack_beam(aug, 0)
    am = np.array([9, 9, 9, 9, 9])
    assert ora.accept_greedy(beams, p["unpack"], am) == (0, 0, [9])
    am = np.array([7, 0, 0, 8, 3])                       # root->7, node(7)->8, node(7,8)->3
    assert ora.accept_greedy(beams, p["unpack"], am) == (2, 1, [7, 8, 3])

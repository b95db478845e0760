"""Shared test helpers: small models as numpy dicts for the oracle."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2403_09919_b200 import synth  # noqa: E402

MICRO = dict(n_layers=2, d_model=64, n_heads=4, d_ffn=172, vocab=128, rms_eps=1e-6,
             rope_theta=10000.0, d_rnn=64, n_head_layers=2, dtype="fp32", max_batch=1,
             max_ctx=96, beam_width=4, beam_length=4, prompt_len=12, steps=8, seed=7)


def micro_model(std=0.25, seed=123, cfg=None):
    """Weights with a larger std than the workloads use, so logits are well separated."""
    cfg = dict(MICRO if cfg is None else cfg)
    w = synth.make_weights(cfg, "cpu", seed=seed, std=std, gain_jitter=0.1)
    W, D = synth.weights_to_numpy(w, cfg)
    return cfg, W, D, w


def first_mismatch(beams, continuation):
    """Closed form for planted beams: per candidate, the index of the first token that differs from the continuation
    (= its accepted length under greedy acceptance when the continuation is the LLM's own greedy stream)."""
    beams = np.asarray(beams)
    cont = np.asarray(continuation[:beams.shape[1]])
    neq = beams != cont[None, :]
    return np.where(neq.any(axis=1), neq.argmax(axis=1), beams.shape[1])


def read_golden(name):
    path = os.path.join(ROOT, "tests", "golden", name)
    with open(path) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------------------- GPU rigs
def dev(a, dtype=None):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda:0", torch.int32 if dtype is None else dtype)


def top2_gap(logits):
    s = np.sort(logits, axis=-1)
    return s[..., -1] - s[..., -2]


class Rig:
    """A model on the GPU (through the C ABI) plus the same stored weight values for the oracle."""

    def __init__(self, name="tiny", flags=0, cfg=None, oracle_dtype=np.float64, std=0.02, **over):
        from oracle import redrafter_oracle as ora
        from paper_2403_09919_b200 import binding
        self.binding = binding
        self.ora = ora
        self.cfg = dict(synth.CONFIGS[name] if cfg is None else cfg, **over)
        self.w = synth.make_weights(self.cfg, "cuda:0", std=std)
        self.W, self.D = synth.weights_to_numpy(self.w, self.cfg)
        self.odt = oracle_dtype
        if oracle_dtype != np.float32:
            self.W, self.D = ora.convert_weights(self.W, self.D, oracle_dtype)
        self.eng = binding.ReDrafter(self.cfg, self.w, flags=flags)
        self.hd = self.cfg["d_model"] // self.cfg["n_heads"]

    def new_kv(self):
        c = self.cfg
        return self.ora.KVCache(c["n_layers"], c["max_ctx"], c["n_heads"], self.hd, self.odt)


# ---------------------------------------------------------------------------- drafter beams under an error bound
def tolerant_beam_search(ora, D, E, g, h, beam_width, beam_length, eps, dtype=np.float64, store=None, cap=6):
    """The oracle's beam search (Section 3.2) with every top-BW decision widened by an error bound.

    An implementation whose cumulative candidate scores are within `eps` of the oracle's must keep candidate c at a
    call if fewer than BW candidates that it can possibly hold reach score(c) - 2 eps ("sure"), and can keep c only if
    fewer than BW candidates that it surely holds exceed score(c) + 2 eps ("maybe").  Candidates descend from the sure
    and maybe beams of the previous call; only descendants of sure beams are surely held.  Returns (sure, maybe,
    widened): two dicts {sequence tuple: oracle score} for the beams after the last call, and the number of calls at
    which some candidate was only "maybe".  The live set may grow to cap x BW beams before the search gives up (None).
    """
    V = D["draft_out"].shape[0]
    E = np.asarray(E, dtype=dtype)
    h = np.asarray(h, dtype=dtype)
    live = [((), 0.0, E[g], True)]              # (sequence, score, state s_t, surely held)
    widened = 0
    for t in range(1, beam_length + 1):
        seqs, vals, states, parent_sure = [], [], [], []
        for (seq, score, s_prev, sure) in live:
            s = s_prev if t == 1 else ora.rnn_cell(D, s_prev, E[seq[-1]], dtype, store)
            lp = ora.log_softmax(ora.draft_head(D, np.concatenate([s, h]), dtype, store))
            # only the best continuations of a beam can be among the best BW of the call; twice that is a safe superset
            top = np.argsort(-lp, kind="stable")[:2 * beam_width + 2]
            for v in top:
                seqs.append(seq + (int(v),)); vals.append(score + lp[v]); states.append(s); parent_sure.append(sure)
        vals = np.array(vals); parent_sure = np.array(parent_sure)
        held = np.sort(vals[parent_sure])[::-1]      # candidates every implementation within eps has
        every = np.sort(vals)[::-1]                  # candidates it may have
        nxt = []
        for i in range(len(vals)):
            can_reach = int((every >= vals[i] - 2 * eps).sum())          # includes the candidate itself
            surely_above = int((held > vals[i] + 2 * eps).sum())
            is_sure = bool(parent_sure[i]) and can_reach <= beam_width
            if is_sure or surely_above < beam_width:
                nxt.append((seqs[i], float(vals[i]), states[i], is_sure))
        if len(nxt) > cap * beam_width:
            return None
        widened += any(not x[3] for x in nxt)
        live = nxt
    sure = {x[0]: x[1] for x in live if x[3]}
    maybe = {x[0]: x[1] for x in live if not x[3]}
    return sure, maybe, widened


def check_beams_within(ora_sets, beams, scores, eps):
    """GPU beams against tolerant_beam_search's result.  Every sure sequence is present, every returned sequence is
    sure or maybe with its score within eps, the sequences are distinct, and the order follows the oracle's scores
    wherever they differ by more than 2 eps.  Returns the number of ranks that were thereby fixed exactly."""
    sure, maybe, _ = ora_sets
    both = dict(maybe); both.update(sure)
    got = [tuple(int(x) for x in b) for b in np.asarray(beams)]
    sc = np.asarray(scores, dtype=np.float64)
    assert len(set(got)) == len(got), "beams are not distinct"
    assert (np.diff(sc) <= 0).all(), "scores are not sorted"
    for s, v in zip(got, sc):
        assert s in both, f"beam {s} cannot be among the best {len(got)} within the error bound"
        assert abs(both[s] - v) <= eps, (s, both[s], v)
    missing = [s for s in sure if s not in got]
    assert not missing, f"beams that every implementation within the bound must return are missing: {missing}"
    true = np.array([both[s] for s in got])
    for i in range(len(got)):
        for j in range(i + 1, len(got)):
            assert true[i] >= true[j] - 2 * eps, (i, j, true[i], true[j])
    # ranks fixed exactly: a sure beam whose oracle score is clear of every other possible beam's by 2 eps
    allv = np.array(sorted(both.values(), reverse=True))
    fixed = 0
    for s in got:
        if s in sure and (np.abs(allv - both[s]) <= 2 * eps).sum() == 1:
            fixed += 1
    return fixed


# ---------------------------------------------------------------------------- logits at a workload's own depth
def row_l2(a, b):
    """Per row: |a - b|_2 / |b|_2."""
    return np.linalg.norm(a - b, axis=-1) / np.linalg.norm(b, axis=-1)


def row_max(a, b):
    """Per row: max |a - b| / max |b|."""
    return np.abs(a - b).max(axis=-1) / np.abs(b).max(axis=-1)


def check_against_storage_noise(got, ref_store, ref_plain, tag, stated=None, l2_factor=1.15, max_factor=1.5):
    """GPU values `got` (rows x features) against the oracle with the path's bf16 storage points (R) and the unrounded
    oracle (U), computed by the caller on the same rows.

    The distance between R and U is the storage noise: what keeping projection inputs, Q, K, V and the softmax weights
    in bf16 costs, measured without any kernel.  It grows as the square root of the depth and passes the stated 3e-2
    at the workloads' own depths.  A correct implementation of the same storage is another sample of that noise: it
    lies as far from U as R does (measured: within 3 % at 2, 32, 40 and 60 layers), and somewhat closer to R, because
    the two samples are partly correlated until a difference in the last bits of an fp32 sum has flipped enough
    roundings downstream (tests/test_oracle_storage.py shows that drift between two CPU runs; measured 0.6-0.7 x R-U at
    32 to 60 layers, 1.0-1.1 x in two-layer models over thousands of keys; sqrt(2) x would be two independent samples).
    So, at any depth:
      mean over the rows of the relative L2 distance  got-U <= l2_factor x R-U,   got-R <= 1.3 x R-U
      worst element over the row's largest magnitude  got-U <= max_factor x R-U,  got-R <= max_factor x R-U.
    An error of 0.4 % per layer in a kernel would raise got-U by more than the 15 % allowed at 32 layers.
    stated: also require the stated tolerance (worst element within `stated` of the row's largest magnitude) against
    both oracles; the depth-reduced cases pass it.  Prints the figures."""
    got, R, U = np.asarray(got, np.float64), np.asarray(ref_store, np.float64), np.asarray(ref_plain, np.float64)
    ru_l2, gu_l2, gr_l2 = row_l2(R, U).mean(), row_l2(got, U).mean(), row_l2(got, R).mean()
    ru_mx, gu_mx, gr_mx = row_max(R, U).max(), row_max(got, U).max(), row_max(got, R).max()
    print(f"{tag}: mean row L2  oracle(bf16 storage) vs oracle {ru_l2:.4f} | GPU vs oracle {gu_l2:.4f} | GPU vs oracle(bf16 storage) {gr_l2:.4f}"
          f"   worst element / row max  {ru_mx:.4f} | {gu_mx:.4f} | {gr_mx:.4f}")
    assert gu_l2 <= l2_factor * ru_l2 and gr_l2 <= 1.3 * ru_l2, (tag, ru_l2, gu_l2, gr_l2)
    assert gu_mx <= max_factor * ru_mx and gr_mx <= max_factor * ru_mx, (tag, ru_mx, gu_mx, gr_mx)
    if stated is not None:
        assert gu_mx < stated and gr_mx < stated, (tag, stated, gu_mx, gr_mx)
    return dict(ru_l2=ru_l2, gu_l2=gu_l2, gr_l2=gr_l2, ru_max=ru_mx, gu_max=gu_mx, gr_max=gr_mx)

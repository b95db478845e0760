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

    def __init__(self, name="tiny", flags=0, cfg=None, oracle_dtype=np.float64, **over):
        from oracle import redrafter_oracle as ora
        from paper_2403_09919_b200 import binding
        self.binding = binding
        self.ora = ora
        self.cfg = dict(synth.CONFIGS[name] if cfg is None else cfg, **over)
        self.w = synth.make_weights(self.cfg, "cuda:0")
        self.W, self.D = synth.weights_to_numpy(self.w, self.cfg)
        self.odt = oracle_dtype
        if oracle_dtype != np.float32:
            self.W, self.D = ora.convert_weights(self.W, self.D, oracle_dtype)
        self.eng = binding.ReDrafter(self.cfg, self.w, flags=flags)
        self.hd = self.cfg["d_model"] // self.cfg["n_heads"]

    def new_kv(self):
        c = self.cfg
        return self.ora.KVCache(c["n_layers"], c["max_ctx"], c["n_heads"], self.hd, self.odt)

"""The counter hand-off between launches changes when a kernel may start, never what it computes.

Two engines with the same seeded weights run the same speculative steps, one with the hand-off (the
default) and one created with RD_CHAIN=0, where every launch waits for its predecessor through the grid
dependency alone.  Everything a step produces must be bit-identical: drafted beams, packed tree,
verification logits, greedy tokens, acceptance, the handed-over state and the KV cache.  A race in the
hand-off (a consumer reading before its producer's last store, a counter reused too early) shows up here
as a difference, and repeating the steps makes it likelier to surface.  Sizes: the depth-reduced 7B shape,
whose launches take the tensor-core path and the two-kernel selection.
"""
import os

import numpy as np
import pytest
import torch

from helpers import Rig
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu


def make_rig(chain):
    cfg = synth.with_layers(dict(synth.CONFIGS["7b"], max_ctx=512), 2)
    old = os.environ.get("RD_CHAIN")
    os.environ["RD_CHAIN"] = "1" if chain else "0"
    try:
        return Rig(cfg=cfg, oracle_dtype=np.float32)
    finally:
        if old is None:
            del os.environ["RD_CHAIN"]
        else:
            os.environ["RD_CHAIN"] = old


def test_hand_off_is_bit_identical_to_grid_dependencies():
    a, b = make_rig(True), make_rig(False)
    rng = np.random.default_rng(5)
    prompts = [rng.integers(0, a.cfg["vocab"], size=150)]
    a.eng.prefill(prompts)
    b.eng.prefill(prompts)
    for sa, sb in zip(a.eng.get_state(), b.eng.get_state()):
        assert torch.equal(sa, sb)
    for step in range(6):
        beams_a, sc_a = a.eng.draft()
        beams_b, sc_b = b.eng.draft()
        assert torch.equal(beams_a, beams_b) and torch.equal(sc_a, sc_b)
        pk_a, pk_b = a.eng.pack(beams_a), b.eng.pack(beams_b)
        assert torch.equal(pk_a.n, pk_b.n) and torch.equal(pk_a.tokens, pk_b.tokens)
        am_a, hid_a, lg_a = a.eng.verify(pk_a, want_logits=True)
        am_b, hid_b, lg_b = b.eng.verify(pk_b, want_logits=True)
        n = int(pk_a.n[0])
        assert torch.equal(lg_a[0, :n], lg_b[0, :n])
        assert torch.equal(hid_a[0, :n], hid_b[0, :n])
        assert torch.equal(am_a, am_b)
        out_a = a.eng.accept(beams_a, pk_a, am_a, hid_a)
        out_b = b.eng.accept(beams_b, pk_b, am_b, hid_b)
        a.eng.poll()
        b.eng.poll()
        assert torch.equal(out_a.n_accept, out_b.n_accept) and torch.equal(out_a.tokens, out_b.tokens)
        for sa, sb in zip(a.eng.get_state(), b.eng.get_state()):
            assert torch.equal(sa, sb)
    assert torch.equal(a.eng.kv_view(), b.eng.kv_view())


def test_fused_steps_repeat_bit_identically():
    """redrafter_step from the same state, twice on each of two engines: four identical token streams."""
    streams = []
    for chain in (True, True, False):
        r = make_rig(chain)
        rng = np.random.default_rng(9)
        r.eng.prefill([rng.integers(0, r.cfg["vocab"], size=97)])
        out = r.binding.AcceptOut(1, r.cfg["beam_length"], "cuda:0")
        toks = []
        for _ in range(8):
            r.eng.step(None, out)
            r.eng.poll()
            toks.append((int(out.n_accept[0]), out.tokens[0].cpu().numpy().copy()))
        streams.append(toks)
    for other in streams[1:]:
        for (na, ta), (nb, tb) in zip(streams[0], other):
            assert na == nb and (ta[:na + 1] == tb[:nb + 1]).all()


def test_a_wait_that_nothing_satisfies_gives_up_and_is_reported():
    """The device-side waits are bounded: one that can never be satisfied returns after about a second, the next
    poll reports RD_ERR_TIMEOUT and clears it, and the engine keeps working."""
    import time
    r = make_rig(True)
    rng = np.random.default_rng(3)
    r.eng.prefill([rng.integers(0, r.cfg["vocab"], size=64)])
    out = r.binding.AcceptOut(1, r.cfg["beam_length"], "cuda:0")
    r.eng.step(None, out)
    r.eng.poll()
    ref_state = [s.clone() for s in r.eng.get_state()]
    t0 = time.time()
    r.eng.selftest_wait()
    with pytest.raises(r.binding.RdError) as e:
        r.eng.poll()
    dt = time.time() - t0
    assert e.value.code == 6 and 0.5 < dt < 10.0          # RD_ERR_TIMEOUT, after the wait's one-second limit
    r.eng.poll()                                          # the status word was cleared
    for a, b in zip(ref_state, r.eng.get_state()):
        assert torch.equal(a, b)                          # nothing of the state was touched
    r.eng.step(None, out)                                 # and the engine still decodes
    r.eng.poll()
    assert int(out.n_accept[0]) >= 0

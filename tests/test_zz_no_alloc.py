"""redrafter_accept_static: the accept step for callers that cannot allocate device memory.

Some users of this library run where nothing may be allocated on the GPU once serving has started
(an allocator-free request loop, a plugin inside a host that owns all device memory).  For them the
library carries the accept step's small scratch inside itself.  This test drives that entry point
through the C ABI next to the ordinary redrafter_accept on an identical second engine, for two
speculative steps in a row, and requires identical results: accepted lengths, best candidates,
emitted tokens, the handed-over state and the compacted KV cache.  It is collected last so that a run
that stops at the first failure has already exercised everything else.
"""
import numpy as np
import pytest
import torch

from helpers import Rig, dev
from paper_2403_09919_b200 import synth

pytestmark = pytest.mark.gpu


def test_accept_static_matches_accept_two_steps_in_a_row():
    cfg = dict(synth.CONFIGS["tiny"], max_batch=2, max_ctx=160)
    a, b = Rig(cfg=cfg), Rig(cfg=cfg)                 # same seeded weights, separate handles and caches
    rng = np.random.default_rng(21)
    prompts = [rng.integers(0, 1024, size=n) for n in (40, 23)]
    a.eng.prefill(prompts)
    b.eng.prefill(prompts)
    for step in range(2):
        beams_a, _ = a.eng.draft()
        beams_b, _ = b.eng.draft()
        assert torch.equal(beams_a, beams_b)
        # make acceptance non-trivial: the first candidate of each sequence starts with the LLM's own token
        am_probe, _, _ = a.eng.verify(a.eng.pack(beams_a))
        b.eng.verify(b.eng.pack(beams_b))            # the same provisional cache rows on both engines
        beams_a[:, 0, 0] = am_probe[:, 0]
        beams_b.copy_(beams_a)
        pk_a, pk_b = a.eng.pack(beams_a), b.eng.pack(beams_b)
        am_a, hid_a, _ = a.eng.verify(pk_a)
        am_b, hid_b, _ = b.eng.verify(pk_b)
        assert torch.equal(am_a, am_b)
        out_a = a.eng.accept(beams_a, pk_a, am_a, hid_a)
        out_b = b.eng.accept_static(beams_b, pk_b, am_b, hid_b)
        a.eng.poll()
        b.eng.poll()
        assert torch.equal(out_a.n_accept, out_b.n_accept) and int(out_a.n_accept.max()) >= 1
        assert torch.equal(out_a.best, out_b.best)
        assert torch.equal(out_a.tokens, out_b.tokens)
        for sa, sb in zip(a.eng.get_state(), b.eng.get_state()):
            assert torch.equal(sa, sb)
        assert torch.equal(a.eng.kv_view(), b.eng.kv_view())


def test_accept_static_rejects_null_arguments():
    r = Rig(cfg=dict(synth.CONFIGS["tiny"]))
    r.eng.prefill([np.arange(8)])
    beams, _ = r.eng.draft()
    pk = r.eng.pack(beams)
    am, hid, _ = r.eng.verify(pk)
    from paper_2403_09919_b200.binding import RdError
    with pytest.raises(RdError) as e:
        r.eng.accept_static(beams, pk, am, None)
    assert e.value.code == 1

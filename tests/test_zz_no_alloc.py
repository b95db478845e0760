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


def test_accept_static_refuses_more_sequences_than_its_scratch_holds():
    """The built-in scratch holds 4096 sequences; a batch of 4097 is refused before anything is enqueued (a caller
    that cannot allocate must learn this from the status code, not from a fault)."""
    from paper_2403_09919_b200.binding import AcceptOut, RdError
    cfg = dict(synth.CONFIGS["tiny"], n_layers=1, d_model=64, n_heads=1, d_ffn=64, vocab=128, d_rnn=64, max_batch=4097,
               max_ctx=8, beam_width=1, beam_length=1)
    r = Rig(cfg=cfg)
    B = 4097
    r.eng.set_state(dev(np.ones(B)), dev(np.zeros(B)), None, batch=B, ctx_bound=1)
    beams = torch.zeros(B, 1, 1, dtype=torch.int32, device="cuda:0")
    pk = r.eng.pack(beams)
    am, hid, _ = r.eng.verify(pk)
    launches = r.eng.launch_count()
    with pytest.raises(RdError) as e:
        r.eng.accept_static(beams, pk, am, hid, AcceptOut(B, 1, "cuda:0"))
    assert e.value.code == 3 and r.eng.launch_count() == launches      # RD_ERR_CAPACITY, nothing enqueued
    r.eng.accept(beams, pk, am, hid)                                      # the workspace-backed entry point takes it
    r.eng.poll()
    # 4096 sequences fit
    r.eng.set_state(dev(np.ones(4096)), dev(np.zeros(4096)), None, batch=4096, ctx_bound=1)
    beams = beams[:4096].contiguous()
    pk = r.eng.pack(beams)
    am, hid, _ = r.eng.verify(pk)
    r.eng.accept_static(beams, pk, am, hid, AcceptOut(4096, 1, "cuda:0"))
    r.eng.poll()

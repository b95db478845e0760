"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from helpers import ROOT
from paper_2403_09919_b200 import binding, build, synth


def _declared():
    text = open(os.path.join(ROOT, "include", "redrafter.h")).read()
    return sorted(set(re.findall(r"RD_API[^;(]*?\b(redrafter_[a-z_]+)\s*\(", text)))


def test_header_symbols_exported():
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert len(names) >= 17
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_sizes_host_only():
    L = binding.lib()
    for name, cfg in synth.CONFIGS.items():
        c = binding.make_config(cfg)
        ws = L.redrafter_workspace_bytes(ctypes.byref(c))
        kv = L.redrafter_kv_bytes(ctypes.byref(c))
        hd = cfg["d_model"] // cfg["n_heads"]
        es = 4 if cfg["dtype"] == "fp32" else 2
        assert kv == cfg["n_layers"] * 2 * cfg["max_batch"] * cfg["n_heads"] * cfg["max_ctx"] * hd * es
        assert ws > 0
    bad = binding.make_config(dict(synth.CONFIGS["tiny"], beam_width=2000))
    assert L.redrafter_workspace_bytes(ctypes.byref(bad)) == 0          # BW > vocab
    bad = binding.make_config(synth.CONFIGS["tiny"])
    bad.struct_bytes = 8
    assert L.redrafter_workspace_bytes(ctypes.byref(bad)) == 0


def test_null_arguments_rejected_without_gpu():
    L = binding.lib()
    assert L.redrafter_init(None, None, None, 0, None, 0, None) == 1
    assert L.redrafter_step(None, None, None, None) == 1
    assert L.redrafter_destroy(None) == 1
    assert L.redrafter_set_sampling(None, 1.0, 0) == 1

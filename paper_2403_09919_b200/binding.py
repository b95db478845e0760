"""ctypes binding of libredrafter.so (include/redrafter.h): argument marshalling only.

Every step of the decode path runs in the library's CUDA kernels; this module turns torch
tensors into device pointers, allocates the caller-owned buffers with torch, and raises on any
non-zero status.  There is no fallback: without the built library, or without a CUDA device,
the calls fail.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

# REDRAFTER_LIB: another build of the same library (a measurement build with extra defines, see build.py)
_LIB_PATH = os.environ.get("REDRAFTER_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libredrafter.so")
_lib = None

RD_DTYPE = {"fp32": 0, "bf16": 1}
RD_FLAG_NO_TREE = 1
RD_FLAG_FORCE_SIMT = 2
STATUS = {0: "RD_OK", 1: "RD_ERR_INVALID_ARG", 2: "RD_ERR_SHAPE", 3: "RD_ERR_CAPACITY", 4: "RD_ERR_STATE",
          5: "RD_ERR_CUDA", 6: "RD_ERR_TIMEOUT", 7: "RD_ERR_UNSUPPORTED"}

EXPORTS = ["redrafter_workspace_bytes", "redrafter_kv_bytes", "redrafter_init", "redrafter_destroy",
           "redrafter_last_error", "redrafter_prefill", "redrafter_draft", "redrafter_pack", "redrafter_verify",
           "redrafter_accept", "redrafter_step", "redrafter_ar_step", "redrafter_get_state", "redrafter_set_state",
           "redrafter_set_ctx_bound", "redrafter_poll", "redrafter_launch_count", "redrafter_profile",
           "redrafter_profile_read", "redrafter_trace", "redrafter_trace_read", "redrafter_trace_bytes",
           "redrafter_accept_static", "redrafter_selftest_wait", "redrafter_set_sampling", "redrafter_route_counts", "redrafter_last_logits", "redrafter_trace_prefetched",
           "redrafter_last_packed_rows"]

ROUTES = ("att_rows16", "att_rows16_shallow", "att_rows64", "att_rows128_tc5", "att_key_split", "att_fp32", "gemm_pairs",
          "gemm_one_cta", "gemm_simt")


class RdConfig(C.Structure):
    _fields_ = [("struct_bytes", C.c_int32), ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("d_ffn", C.c_int32), ("vocab", C.c_int32), ("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("d_rnn", C.c_int32), ("n_head_layers", C.c_int32), ("dtype", C.c_int32), ("max_batch", C.c_int32),
                ("max_ctx", C.c_int32), ("beam_width", C.c_int32), ("beam_length", C.c_int32), ("flags", C.c_uint32)]


class RdWeights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p),
                ("attn_norm", C.POINTER(C.c_void_p)), ("wqkv", C.POINTER(C.c_void_p)), ("wo", C.POINTER(C.c_void_p)),
                ("ffn_norm", C.POINTER(C.c_void_p)), ("w_gate_up", C.POINTER(C.c_void_p)),
                ("w_down", C.POINTER(C.c_void_p)), ("rnn_u", C.c_void_p), ("rnn_w", C.c_void_p), ("rnn_b", C.c_void_p),
                ("head_w", C.POINTER(C.c_void_p)), ("head_b", C.POINTER(C.c_void_p)), ("draft_out", C.c_void_p)]


class RdPacked(C.Structure):
    _fields_ = [("tokens", C.c_void_p), ("n", C.c_void_p), ("unpack", C.c_void_p), ("pos", C.c_void_p),
                ("mask", C.c_void_p), ("parent", C.c_void_p)]


class RdAcceptOut(C.Structure):
    _fields_ = [("n_accept", C.c_void_p), ("best", C.c_void_p), ("tokens", C.c_void_p)]


def lib():
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2403_09919_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(_LIB_PATH)
        vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
        L.redrafter_workspace_bytes.restype = sz
        L.redrafter_workspace_bytes.argtypes = [C.POINTER(RdConfig)]
        L.redrafter_kv_bytes.restype = sz
        L.redrafter_kv_bytes.argtypes = [C.POINTER(RdConfig)]
        L.redrafter_init.argtypes = [C.POINTER(RdConfig), C.POINTER(RdWeights), vp, sz, vp, sz, C.POINTER(vp)]
        L.redrafter_destroy.argtypes = [vp]
        L.redrafter_last_error.restype = C.c_char_p
        L.redrafter_last_error.argtypes = [vp]
        L.redrafter_prefill.argtypes = [vp, vp, vp, i32, i32, vp]
        L.redrafter_draft.argtypes = [vp, vp, vp, vp]
        L.redrafter_pack.argtypes = [vp, vp, vp, C.POINTER(RdPacked)]
        L.redrafter_verify.argtypes = [vp, C.POINTER(RdPacked), vp, vp, vp, vp]
        L.redrafter_accept.argtypes = [vp, vp, C.POINTER(RdPacked), vp, vp, vp, C.POINTER(RdAcceptOut)]
        L.redrafter_accept_static.argtypes = [vp, vp, C.POINTER(RdPacked), vp, vp, vp, C.POINTER(RdAcceptOut)]
        L.redrafter_step.argtypes = [vp, vp, vp, C.POINTER(RdAcceptOut)]
        L.redrafter_ar_step.argtypes = [vp, vp, vp]
        L.redrafter_get_state.argtypes = [vp, vp, vp, vp, vp]
        L.redrafter_set_state.argtypes = [vp, vp, vp, vp, vp, i32]
        L.redrafter_set_ctx_bound.argtypes = [vp, i32]
        L.redrafter_set_sampling.argtypes = [vp, C.c_float, C.c_uint64]
        L.redrafter_poll.argtypes = [vp, vp]
        L.redrafter_launch_count.restype = C.c_int64
        L.redrafter_launch_count.argtypes = [vp]
        L.redrafter_profile.argtypes = [vp, C.c_int]
        L.redrafter_profile_read.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                             C.POINTER(C.c_int64)]
        L.redrafter_trace.argtypes = [vp, C.c_int, vp]
        L.redrafter_trace_read.argtypes = [vp, vp, vp, i32]
        L.redrafter_trace_bytes.argtypes = [vp, vp, i32]
        L.redrafter_selftest_wait.argtypes = [vp, vp]
        L.redrafter_last_logits.argtypes = [vp, vp, vp, i32]
        L.redrafter_trace_prefetched.argtypes = [vp, vp, i32]
        L.redrafter_last_packed_rows.argtypes = [vp, vp, vp]
        L.redrafter_route_counts.argtypes = [vp, C.POINTER(C.c_int64), i32]
        _lib = L
    return _lib


def make_config(cfg, flags=0):
    c = RdConfig()
    c.struct_bytes = C.sizeof(RdConfig)
    for k in ("n_layers", "d_model", "n_heads", "d_ffn", "vocab", "d_rnn", "n_head_layers", "max_batch", "max_ctx",
              "beam_width", "beam_length"):
        setattr(c, k, int(cfg[k]))
    c.rms_eps = float(cfg["rms_eps"])
    c.rope_theta = float(cfg["rope_theta"])
    c.dtype = RD_DTYPE[cfg["dtype"]]
    c.flags = int(flags)
    return c


class RdError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{STATUS.get(code, code)}: {msg}")
        self.code = code


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Packed:
    """Caller-owned device buffers of one rd_packed."""

    def __init__(self, B, BW, L, device):
        nmax = 1 + BW * L
        mw = (nmax + 31) // 32
        i32 = dict(dtype=torch.int32, device=device)
        self.tokens = torch.zeros(B, nmax, **i32)
        self.n = torch.zeros(B, **i32)
        self.unpack = torch.zeros(B, BW, L + 1, **i32)
        self.pos = torch.zeros(B, nmax, **i32)
        self.mask = torch.zeros(B, nmax, mw, **i32)      # bit pattern of uint32
        self.parent = torch.zeros(B, nmax, **i32)
        self.c = RdPacked(*[t.data_ptr() for t in (self.tokens, self.n, self.unpack, self.pos, self.mask, self.parent)])

    def mask_bool(self, b):
        """[n, n] boolean tree mask of sequence b (host)."""
        n = int(self.n[b])
        words = self.mask[b, :n].cpu().numpy().view("uint32")
        import numpy as np
        bits = ((words[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1).reshape(n, -1)
        return bits[:, :n].astype(bool)


class AcceptOut:
    def __init__(self, B, L, device):
        i32 = dict(dtype=torch.int32, device=device)
        self.n_accept = torch.zeros(B, **i32)
        self.best = torch.zeros(B, **i32)
        self.tokens = torch.zeros(B, L + 1, **i32)
        self.c = RdAcceptOut(self.n_accept.data_ptr(), self.best.data_ptr(), self.tokens.data_ptr())


class ReDrafter:
    """A handle plus the device buffers it borrows (KV cache, workspace), allocated with torch."""

    def __init__(self, cfg, weights, device="cuda:0", flags=0):
        if not torch.cuda.is_available():
            raise RuntimeError("ReDrafter needs a CUDA device; there is no CPU path")
        self.L = lib()
        self.cfg = dict(cfg)
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.c_cfg = make_config(cfg, flags)
        self.weights = weights                      # keep the tensors alive
        want = torch.float32 if cfg["dtype"] == "fp32" else torch.bfloat16
        for k, t in weights.items():
            if t.dtype != want or not t.is_cuda or not t.is_contiguous():
                raise ValueError(f"weight {k}: expected contiguous {want} on a CUDA device")
        nl, nh = cfg["n_layers"], cfg["n_head_layers"]

        def arr(prefix, n):
            return (C.c_void_p * n)(*[weights[f"{prefix}.{l}"].data_ptr() for l in range(n)])

        self._arrays = {k: arr(k, nl) for k in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down")}
        self._arrays.update({k: arr(k, nh) for k in ("head_w", "head_b")})
        w = RdWeights()
        for k in ("tok_emb", "final_norm", "lm_head", "rnn_u", "rnn_w", "rnn_b", "draft_out"):
            setattr(w, k, weights[k].data_ptr())
        for k, a in self._arrays.items():
            setattr(w, k, C.cast(a, C.POINTER(C.c_void_p)))
        self.c_w = w
        ws_bytes = self.L.redrafter_workspace_bytes(C.byref(self.c_cfg))
        kv_bytes = self.L.redrafter_kv_bytes(C.byref(self.c_cfg))
        if ws_bytes == 0:
            raise RdError(2, "config rejected by redrafter_workspace_bytes")
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)
        self.kv = torch.zeros(kv_bytes, dtype=torch.uint8, device=self.device)
        self.ws_bytes, self.kv_bytes = ws_bytes, kv_bytes
        torch.cuda.synchronize()
        hp = C.c_void_p()
        rc = self.L.redrafter_init(C.byref(self.c_cfg), C.byref(w), self.kv.data_ptr(), kv_bytes,
                                   self.workspace.data_ptr(), ws_bytes, C.byref(hp))
        if rc:
            raise RdError(rc, "redrafter_init failed: " + self.L.redrafter_last_error(None).decode())
        self.h = hp
        self.B = cfg["max_batch"]
        self.BW, self.Lb, self.d, self.V = cfg["beam_width"], cfg["beam_length"], cfg["d_model"], cfg["vocab"]
        self.nmax = 1 + self.BW * self.Lb

    def close(self):
        if getattr(self, "h", None):
            self.L.redrafter_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ck(self, rc):
        if rc:
            raise RdError(rc, self.L.redrafter_last_error(self.h).decode())

    # ---- the C-ABI calls, same names ----
    def prefill(self, prompts):
        """prompts: list of 1-D int sequences (host)."""
        import numpy as np
        B = len(prompts)
        mp = max(len(p) for p in prompts)
        tok = np.zeros((B, mp), dtype=np.int32)
        ln = np.zeros(B, dtype=np.int32)
        for b, p in enumerate(prompts):
            tok[b, :len(p)] = np.asarray(p, dtype=np.int32)
            ln[b] = len(p)
        self.B = B
        self._ck(self.L.redrafter_prefill(self.h, tok.ctypes.data, ln.ctypes.data, mp, B, _stream()))

    def draft(self, beams=None, scores=None):
        beams = torch.empty(self.B, self.BW, self.Lb, dtype=torch.int32, device=self.device) if beams is None else beams
        scores = torch.empty(self.B, self.BW, dtype=torch.float32, device=self.device) if scores is None else scores
        self._ck(self.L.redrafter_draft(self.h, _stream(), _ptr(beams), _ptr(scores)))
        return beams, scores

    def pack(self, beams, out=None):
        out = Packed(self.B, self.BW, self.Lb, self.device) if out is None else out
        self._ck(self.L.redrafter_pack(self.h, _ptr(beams), _stream(), C.byref(out.c)))
        return out

    def verify(self, packed, want_hidden=True, want_logits=False):
        argmax = torch.empty(self.B, self.nmax, dtype=torch.int32, device=self.device)
        hidden = torch.zeros(self.B, self.nmax, self.d, dtype=torch.float32, device=self.device) if want_hidden else None
        logits = torch.zeros(self.B, self.nmax, self.V, dtype=torch.float32, device=self.device) if want_logits else None
        self._ck(self.L.redrafter_verify(self.h, C.byref(packed.c), _stream(), _ptr(argmax), _ptr(hidden), _ptr(logits)))
        return argmax, hidden, logits

    def accept(self, beams, packed, argmax, hidden, out=None):
        out = AcceptOut(self.B, self.Lb, self.device) if out is None else out
        self._ck(self.L.redrafter_accept(self.h, _ptr(beams), C.byref(packed.c), _ptr(argmax), _ptr(hidden), _stream(),
                                         C.byref(out.c)))
        return out

    def accept_static(self, beams, packed, argmax, hidden, out=None):
        """redrafter_accept_static: the accept step with its scratch inside the library (no allocation)."""
        out = AcceptOut(self.B, self.Lb, self.device) if out is None else out
        self._ck(self.L.redrafter_accept_static(self.h, _ptr(beams), C.byref(packed.c), _ptr(argmax), _ptr(hidden),
                                                _stream(), C.byref(out.c)))
        return out

    def step(self, planted_beams=None, out=None):
        self._ck(self.L.redrafter_step(self.h, _ptr(planted_beams), _stream(), C.byref(out.c) if out is not None else None))
        return out

    def ar_step(self, token=None):
        self._ck(self.L.redrafter_ar_step(self.h, _stream(), _ptr(token)))
        return token

    def set_sampling(self, temperature, seed=0):
        """temperature > 0: the LLM's tokens are draws keyed by (seed; sequence, position); 0: greedy."""
        self._ck(self.L.redrafter_set_sampling(self.h, float(temperature), int(seed)))

    def get_state(self):
        ctx = torch.empty(self.B, dtype=torch.int32, device=self.device)
        root = torch.empty(self.B, dtype=torch.int32, device=self.device)
        h = torch.empty(self.B, self.d, dtype=torch.float32, device=self.device)
        self._ck(self.L.redrafter_get_state(self.h, _stream(), _ptr(ctx), _ptr(root), _ptr(h)))
        return ctx, root, h

    def set_ctx_bound(self, bound):
        self._ck(self.L.redrafter_set_ctx_bound(self.h, int(bound)))

    def set_state(self, ctx=None, root=None, h=None, batch=None, ctx_bound=None):
        batch = self.B if batch is None else batch
        self._ck(self.L.redrafter_set_state(self.h, _stream(), _ptr(ctx), _ptr(root), _ptr(h), batch))
        self.B = batch
        if ctx_bound is not None:
            self._ck(self.L.redrafter_set_ctx_bound(self.h, int(ctx_bound)))

    def selftest_wait(self):
        self._ck(self.L.redrafter_selftest_wait(self.h, _stream()))

    def poll(self):
        self._ck(self.L.redrafter_poll(self.h, _stream()))

    def profile(self, enable):
        self._ck(self.L.redrafter_profile(self.h, 1 if enable else 0))

    def profile_read(self, cls):
        """(ms, bytes, launches) summed since profile(True) for class 0 (projections) or 1 (attention)."""
        ms, by, n = C.c_double(), C.c_double(), C.c_int64()
        self._ck(self.L.redrafter_profile_read(self.h, cls, C.byref(ms), C.byref(by), C.byref(n)))
        return ms.value, by.value, n.value

    def trace(self, enable):
        self._ck(self.L.redrafter_trace(self.h, 1 if enable else 0, _stream()))

    def trace_read(self, max_launches=512):
        """[n, 8] uint64 %globaltimer records of the traced projection launches (host numpy array)."""
        import numpy as np
        buf = np.zeros((max_launches, 8), dtype=np.uint64)
        n = self.L.redrafter_trace_read(self.h, _stream(), buf.ctypes.data, max_launches)
        if n < 0:
            self._ck(-n)
        return buf[:n]

    def trace_bytes(self, max_launches=512):
        """Weight bytes of each traced launch (0 for launches that are not projections)."""
        import numpy as np
        buf = np.zeros(max_launches, dtype=np.float64)
        n = self.L.redrafter_trace_bytes(self.h, buf.ctypes.data, max_launches)
        if n < 0:
            self._ck(-n)
        return buf[:n]

    def last_logits(self, rows):
        """[rows, V] fp32 logits of the last forward pass (device tensor)."""
        out = torch.empty(rows, self.V, dtype=torch.float32, device=self.device)
        self._ck(self.L.redrafter_last_logits(self.h, _stream(), _ptr(out), rows))
        return out

    def route_counts(self):
        """Launches per kernel variant since the handle was made: dict keyed by ROUTES."""
        buf = (C.c_int64 * len(ROUTES))()
        self._ck(self.L.redrafter_route_counts(self.h, buf, len(ROUTES)))
        return dict(zip(ROUTES, list(buf)))

    def trace_prefetched(self, max_launches=512):
        """Of trace_bytes, the bytes each projection launch requests before its dependency wait."""
        import numpy as np
        buf = np.zeros(max_launches, dtype=np.float64)
        n = self.L.redrafter_trace_prefetched(self.h, buf.ctypes.data, max_launches)
        if n < 0:
            self._ck(-n)
        return buf[:n]

    def last_packed_rows(self, out=None):
        """[B] int32 packed rows per sequence of the most recent step (device tensor)."""
        out = torch.empty(self.B, dtype=torch.int32, device=self.device) if out is None else out
        self._ck(self.L.redrafter_last_packed_rows(self.h, _stream(), _ptr(out)))
        return out

    def launch_count(self):
        return int(self.L.redrafter_launch_count(self.h))

    def kv_view(self):
        """The KV cache as a tensor [n_layers, 2, max_batch, n_heads, max_ctx, head_dim]."""
        c = self.cfg
        dt = torch.float32 if c["dtype"] == "fp32" else torch.bfloat16
        hd = c["d_model"] // c["n_heads"]
        return self.kv.view(dt).view(c["n_layers"], 2, c["max_batch"], c["n_heads"], c["max_ctx"], hd)

"""Benchmark of one ReDrafter speculative decode step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 7b] [--impl ours|reference]

A step is one pass of the whole hot path (draft -> pack -> verify -> accept) for one batch; the
default workload is the Vicuna-7B-shaped bs1 configuration.  Prints ONE JSON line.

Two side modes print one JSON line per point and a table on stderr instead: `--sweep` (beam width x
batch at the workload's layer shapes) and `--prefill` (prompt processing).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2403_09919_b200 import synth  # noqa: E402

METRIC = "decode tokens/s (7B-shape, bs1)"
UNIT = "tokens/s"


# --------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def step_bytes(cfg, ctx, n_rows=None):
    """Algorithmic bytes one step must read: LLM weights once, drafter weights once per call
    (head on each of the L calls, RNN on L-1), KV cache of the context once."""
    es = 4 if cfg["dtype"] == "fp32" else 2
    d, Fd, V, L = cfg["d_model"], cfg["d_ffn"], cfg["vocab"], cfg["beam_length"]
    dh = cfg["d_rnn"] + d
    per_layer = 4 * d * d + 3 * d * Fd
    llm = cfg["n_layers"] * per_layer + V * d
    head = cfg["n_head_layers"] * dh * dh + V * dh
    rnn = cfg["d_rnn"] * (cfg["d_rnn"] + d)
    kv = cfg["n_layers"] * 2 * d * ctx
    return dict(llm=llm * es, drafter=(L * head + (L - 1) * rnn) * es, kv=kv * es,
                total=(llm + L * head + (L - 1) * rnn + kv) * es, ar=(llm + kv) * es)


# --------------------------------------------------------------------------- CPU oracle legs
def host_weights(cfg):
    """The workload's seeded weights as host fp32 arrays for the oracle.  Drawn on the GPU when there is one (the same
    generator and seeds the CUDA arm uses, seconds instead of minutes for 7 G values) and copied to the host, else on
    the CPU.  Input generation only: none of the library's kernels is involved."""
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    w = synth.make_weights(cfg, dev)
    W, D = synth.weights_to_numpy(w, cfg)
    del w
    if dev != "cpu":
        torch.cuda.empty_cache()
    return W, D


class OracleFull:
    """The oracle, as it stands, on the workload itself: all layers, its own prefill of the workload's prompt (untimed,
    like the CUDA arm's), then whole speculative steps timed one by one.  fp32 numpy, batch 1."""

    def __init__(self, cfg, sampling=None, weights=None):
        from oracle import redrafter_oracle as ora
        self.ora, self.cfg, self.sampling = ora, cfg, sampling
        self.W, self.D = weights if weights is not None else host_weights(cfg)
        self.prompt = synth.make_prompts(cfg, 1, seed=cfg.get("seed", 0))[0]
        self.extrapolated = False

    def run(self, steps, warmup=0):
        ora, cfg = self.ora, self.cfg
        BW, L = cfg["beam_width"], cfg["beam_length"]
        hd = cfg["d_model"] // cfg["n_heads"]
        cap = len(self.prompt) + (steps + warmup) * (L + 1) + 2 + BW * L
        kv = ora.KVCache(cfg["n_layers"], cap, cfg["n_heads"], hd, np.float32)
        t0 = time.perf_counter()
        ctx, g, h = ora.prefill(self.W, cfg, self.prompt, kv, np.float32, self.sampling)
        prefill_s = time.perf_counter() - t0
        tot_s, tot_tok, rows = 0.0, 0, 0
        for s in range(warmup + steps):
            t0 = time.perf_counter()
            r = ora.spec_step(self.W, self.D, cfg, kv, ctx, g, h, BW, L, dtype=np.float32, sampling=self.sampling)
            dt = time.perf_counter() - t0
            ctx, g, h = r["ctx"], r["g"], r["h"]
            if s >= warmup:
                tot_s += dt; tot_tok += len(r["emitted"]); rows += int(r["packed"]["n"])
        sample = (f"{steps} whole oracle steps of the workload itself ({cfg['n_layers']} layers, fp32 numpy) after {warmup} warm-up, "
                  f"on the cache its own prefill of the {len(self.prompt)}-token prompt wrote ({prefill_s:.0f} s, untimed); drafter's own "
                  f"beams, mean {rows / steps:.0f} packed rows; {tot_s:.1f} s of timed CPU work")
        return dict(value=tot_tok / tot_s, ms_per_step=1e3 * tot_s / steps, sample=sample, timed_s=tot_s)


class OracleSample:
    """For the workloads whose full-depth oracle step takes minutes (13B, batched 7B, 33B): the oracle on a
    depth-reduced copy, full per-layer shapes, `sample_layers` layers, fp32 numpy.  One step is timed in parts and
    EXTRAPOLATED to the full depth: t_step = t_draft + t_pack + (n_layers / sample_layers) * t_layers + t_lm_head + t_accept."""

    def __init__(self, cfg, sample_layers=2, sampling=None):
        self.cfg = cfg
        self.sampling = sampling
        self.sample_layers = min(sample_layers, cfg["n_layers"])
        self.c = synth.with_layers(cfg, self.sample_layers)
        w = synth.make_weights(self.c, "cpu")
        self.W, self.D = synth.weights_to_numpy(w, self.c)
        self.extrapolated = True

    def step(self, seed=0):
        from oracle import redrafter_oracle as ora
        cfg, c, W, D = self.cfg, self.c, self.W, self.D
        dt = np.float32
        BW, L = cfg["beam_width"], cfg["beam_length"]
        rng = np.random.default_rng(seed)
        hd = c["d_model"] // c["n_heads"]
        ctx = cfg["prompt_len"] if isinstance(cfg["prompt_len"], int) else cfg["prompt_len"][1]
        kv = ora.KVCache(c["n_layers"], ctx + 1 + BW * L, c["n_heads"], hd, dt)
        kv.k[:, :ctx] = rng.normal(size=kv.k[:, :ctx].shape).astype(dt)      # a filled cache of the right size
        kv.v[:, :ctx] = rng.normal(size=kv.v[:, :ctx].shape).astype(dt)
        g = int(rng.integers(0, c["vocab"]))
        h = rng.normal(size=c["d_model"]).astype(dt)
        t0 = time.perf_counter()
        beams, _ = ora.beam_search(D, W["tok_emb"], g, h, BW, L, dt)
        t1 = time.perf_counter()
        aug = np.concatenate([np.full((BW, 1), g), beams], axis=1)
        p = ora.pack_beam(aug, ctx)
        t2 = time.perf_counter()
        hidden, _ = ora.llm_forward(W, c, p["tokens"], p["pos"], p["mask"], kv, ctx, dt, want_logits=False)
        t3 = time.perf_counter()
        logits = hidden @ W["lm_head"].T
        am = ora.choose_rows(logits, p["pos"], self.sampling)
        t4 = time.perf_counter()
        a, best, emitted = ora.accept_greedy(beams, p["unpack"], am)
        ora.compact_kv(kv, ctx, p["unpack"], best, a)
        t5 = time.perf_counter()
        scale = cfg["n_layers"] / self.sample_layers
        full = (t1 - t0) + (t2 - t1) + scale * (t3 - t2) + (t4 - t3) + (t5 - t4)
        return dict(step_s=full, tokens=len(emitted), cpu_s=t5 - t0, rows=int(p["n"]))

    def run(self, steps, warmup=0):
        for s in range(warmup):
            self.step(1000 + s)
        tot_s, tot_tok, cpu_s, rows = 0.0, 0, 0.0, 0
        for s in range(steps):
            r = self.step(s)
            tot_s += r["step_s"]; tot_tok += r["tokens"]; cpu_s += r["cpu_s"]; rows += r["rows"]
        sample = (f"EXTRAPOLATED: {steps} oracle steps on a {self.sample_layers}-layer copy of the workload at full per-layer "
                  f"shapes (fp32 numpy, filled cache of {self.cfg['prompt_len']} tokens, drafter's own beams, one sequence, mean "
                  f"{rows / steps:.0f} packed rows); the layer time is scaled by n_layers/{self.sample_layers}; {cpu_s:.1f} s of CPU work")
        return dict(value=tot_tok / tot_s, ms_per_step=1e3 * tot_s / steps, sample=sample, timed_s=cpu_s)


def oracle_leg(args, cfg):
    """The full-depth oracle where a step takes seconds (tiny, 7B bs1); the depth-reduced, extrapolated sample elsewhere."""
    full = cfg["max_batch"] == 1 and cfg["n_layers"] * cfg["d_model"] <= 32 * 4096 and not args.oracle_sample
    return OracleFull(cfg, oracle_sampling(args)) if full else OracleSample(cfg, args.oracle_layers, oracle_sampling(args))


def oracle_sampling(args):
    return dict(temperature=args.temperature, seed=args.sample_seed) if args.temperature > 0 else None


def cpu_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args, cfg):
    """--impl reference: the oracle, as it stands, on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, args.reference_max_steps))
    warm = min(args.warmup, 1)
    leg = oracle_leg(args, cfg)
    r = leg.run(steps, warmup=warm)
    value, sample = r["value"], r["sample"]
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warm, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(args, cfg),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle", "sample": sample,
                             "extrapolated": leg.extrapolated},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    if not leg.extrapolated:
        line["ms_per_step"] = r["ms_per_step"]      # a measured step time; an extrapolated one is not reported as such
    print(json.dumps(line))


def workload_config(args, cfg):
    return {"workload": f"{args.workload}: {cfg['n_layers']} layers d={cfg['d_model']} heads={cfg['n_heads']} ffn={cfg['d_ffn']} "
                        f"vocab={cfg['vocab']} {cfg['dtype']}, batch {cfg['max_batch']}, prompt {cfg['prompt_len']} uniform-random "
                        f"tokens, beam width {cfg['beam_width']}, beam length {cfg['beam_length']}, "
                        + (f"acceptance against the LLM's own draws at temperature {args.temperature}" if args.temperature > 0
                           else "greedy acceptance") + ", random-init weights",
            "beams": "drafter's own (random-init drafter and LLM are uncorrelated: about 1 token per step by construction)",
            "l2": "inputs larger than L2: every step streams all weights (>= 13 GB at 7B) so nothing is reused from the 126 MB L2",
            "parallelism": "replicas only (no collective)"}


# --------------------------------------------------------------------------- replicas (N > 1)
def reduce_over_ranks(ms, tokens, device):
    """Whole-job figures of N independent replicas: the slowest rank's time and the sum of the tokens.
    No-op without an initialised process group.  Works on any backend (tests run it over gloo)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return ms, tokens
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    tk = torch.tensor([tokens], device=device, dtype=torch.int64)
    dist.all_reduce(tk, op=dist.ReduceOp.SUM)
    return float(t.item()), int(tk.item())


def shard_of_rank(rank):
    """Replicas share nothing: each rank decodes its own prompts (seed offset) with its own copy of the weights."""
    return {"prompt_seed_offset": 100 * rank}


# --------------------------------------------------------------------------- GPU legs
def packed_rows_summary(n, BW, L):
    """Packed rows per sequence and step (root + deduplicated draft tokens) against the 1 + BW * L rows the flat layout
    would verify: the synthetic analogue of Figure 5 (left)."""
    n = np.asarray(n).reshape(-1)
    flat = 1 + BW * L
    edges = np.linspace(0, flat, 9).round().astype(int)
    hist, _ = np.histogram(n, bins=edges)
    return {"flat_rows": flat, "mean": float(n.mean()), "min": int(n.min()), "max": int(n.max()),
            "reduction": float(1.0 - n.mean() / flat), "histogram": {f"{edges[i] + (i > 0)}-{edges[i + 1]}": int(hist[i]) for i in range(8)},
            "first_steps": [int(x) for x in n[:16]]}


def timed_loop(eng, n, fn):
    """n calls of fn between two events on the current stream; returns ms."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(n):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def run_sweep(args, cfg):
    """Beam width x batch sweep at the workload's layer shapes (Section 4.2's trade-off on synthetic shapes): where a
    step stops being a weight stream and becomes tensor-core work.  One line of JSON per point and a table on stderr.
    Not part of the default run."""
    from paper_2403_09919_b200 import binding
    device = "cuda:0"
    torch.cuda.set_device(device)
    peak_bw, _ = measured_peaks()
    peak_tf = 1411.0
    try:
        with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "MEASURED_PEAKS.json")) as f:
            peak_tf = float(json.load(f).get("bf16_tflops_sustained", peak_tf))
    except Exception:
        pass
    w = synth.make_weights(cfg, device)
    L = cfg["beam_length"]
    rows = []
    for BW in [int(x) for x in args.sweep_bw.split(",")]:
        for B in [int(x) for x in args.sweep_batch.split(",")]:
            c = dict(cfg, beam_width=BW, max_batch=B, prompt_len=args.sweep_prompt)
            need = args.warmup + args.steps
            c["max_ctx"] = args.sweep_prompt + (need + 2) * (L + 1) + 2 + BW * L
            eng = binding.ReDrafter(c, w, device=device, flags=binding.RD_FLAG_NO_TREE if args.flat else 0)
            prompts = synth.make_prompts(c, B, seed=c.get("seed", 0))
            out = binding.AcceptOut(B, L, device)
            eng.prefill(prompts)
            beams, _ = eng.draft()
            n_rows = int(eng.pack(beams).n.sum().item())       # rows of a typical step (the drafter's own beams)
            for _ in range(args.warmup):
                eng.step(None, out)

            def one(i):
                eng.step(None, out)
            ms = timed_loop(eng, args.steps, one) / args.steps
            eng.poll()
            ctx = args.sweep_prompt + (args.warmup + args.steps / 2) * 1.0
            sb = step_bytes(c, ctx * B)
            es = 2
            flops = 2.0 * n_rows * (sb["llm"] / es) + 2.0 * (B * BW) * (sb["drafter"] / es) + 4.0 * n_rows * ctx * c["d_model"] * c["n_layers"]
            t_bw, t_tc = sb["total"] / (peak_bw * 1e9) * 1e3, flops / (peak_tf * 1e12) * 1e3
            row = {"sweep": True, "tree_attention": not args.flat, "beam_width": BW, "batch": B, "packed_rows": n_rows, "ms_per_step": ms,
                   "algorithmic_gb": sb["total"] / 1e9, "dense_tflop": flops / 1e12, "hbm_bound_ms": t_bw, "tensor_bound_ms": t_tc,
                   "roofline_ms": max(t_bw, t_tc), "frac_of_roofline": max(t_bw, t_tc) / ms,
                   "bound": "hbm" if t_bw >= t_tc else "tensor"}
            rows.append(row)
            print(json.dumps(row), flush=True)
            eng.close()
            del eng
    print("| BW | batch | packed rows | ms/step | HBM-bound ms | tensor-bound ms | bound | roofline frac |", file=sys.stderr)
    print("|---|---|---|---|---|---|---|---|", file=sys.stderr)
    for r in rows:
        print("| %d | %d | %d | %.2f | %.2f | %.2f | %s | %.2f |" % (r["beam_width"], r["batch"], r["packed_rows"], r["ms_per_step"],
              r["hbm_bound_ms"], r["tensor_bound_ms"], r["bound"], r["frac_of_roofline"]), file=sys.stderr)


def run_prefill(args, cfg):
    """Prompt processing (the pass that precedes the decode loop) at the workload's layer shapes: many rows per launch,
    causal attention.  One line of JSON per (batch, prompt length) and a table on stderr.  Not part of the default run."""
    from paper_2403_09919_b200 import binding
    device = "cuda:0"
    torch.cuda.set_device(device)
    peak_bw, _ = measured_peaks()
    peak_tf = 1411.0
    try:
        with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "MEASURED_PEAKS.json")) as f:
            peak_tf = float(json.load(f).get("bf16_tflops_sustained", peak_tf))
    except Exception:
        pass
    w = synth.make_weights(cfg, device)
    es = 2
    rows = []
    for B in [int(x) for x in args.prefill_batch.split(",")]:
        for P in [int(x) for x in args.prefill_len.split(",")]:
            c = dict(cfg, max_batch=B, prompt_len=P)
            c["max_ctx"] = P + 2 * (c["beam_length"] + 1) + 2 + c["beam_width"] * c["beam_length"]
            eng = binding.ReDrafter(c, w, device=device)
            prompts = synth.make_prompts(c, B, seed=c.get("seed", 0))
            reps = 3
            eng.prefill(prompts)                      # warm-up
            ms = timed_loop(eng, reps, lambda i: eng.prefill(prompts)) / reps
            eng.poll()
            sb = step_bytes(c, 0)
            n_tok = B * P
            cap = max(1024, B * (1 + c["beam_width"] * c["beam_length"]))      # rows one pass holds
            passes = (n_tok + cap - 1) // cap
            flops = 2.0 * n_tok * (sb["llm"] / es) + 4.0 * B * (P * (P + 1) / 2) * c["d_model"] * c["n_layers"]
            t_bw, t_tc = passes * sb["llm"] / (peak_bw * 1e9) * 1e3, flops / (peak_tf * 1e12) * 1e3
            row = {"prefill": True, "batch": B, "prompt_len": P, "tokens": n_tok, "passes": passes, "rows_per_pass": cap,
                   "ms": ms, "tokens_per_s": n_tok / ms * 1e3, "dense_tflop": flops / 1e12, "tflops": flops / ms / 1e9,
                   "weight_stream_ms": t_bw, "tensor_bound_ms": t_tc, "frac_of_roofline": max(t_bw, t_tc) / ms}
            rows.append(row)
            print(json.dumps(row), flush=True)
            eng.close()
            del eng
    print("| batch | prompt | tokens | passes x rows | ms | tokens/s | TFLOP/s | weight-stream ms | tensor-bound ms | roofline frac |", file=sys.stderr)
    print("|---|---|---|---|---|---|---|---|---|---|", file=sys.stderr)
    for r in rows:
        print("| %d | %d | %d | %d x %d | %.2f | %.0f | %.0f | %.2f | %.2f | %.2f |" % (r["batch"], r["prompt_len"], r["tokens"], r["passes"],
              r["rows_per_pass"], r["ms"], r["tokens_per_s"], r["tflops"], r["weight_stream_ms"], r["tensor_bound_ms"],
              r["frac_of_roofline"]), file=sys.stderr)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="7b", choices=sorted(synth.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="depth-reduced run (0 = the workload's depth)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--oracle-layers", type=int, default=2)
    ap.add_argument("--reference-max-steps", type=int, default=3)
    ap.add_argument("--cpu-steps", type=int, default=3)
    ap.add_argument("--oracle-sample", action="store_true", help="time the depth-reduced oracle sample even where the full oracle is affordable")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the planted-beam and autoregressive comparison legs")
    ap.add_argument("--sweep", action="store_true", help="beam width x batch sweep instead of the benchmark line")
    ap.add_argument("--sweep-bw", default="1,4,8,16,32")
    ap.add_argument("--sweep-batch", default="1,2,4,8,16")
    ap.add_argument("--sweep-prompt", type=int, default=256)
    ap.add_argument("--flat", action="store_true", help="sweep without dynamic tree attention: every candidate sends all its tokens")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="> 0: the LLM's tokens are draws (Gumbel-max, counter-based noise) instead of greedy; the paper's "
                         "headline numbers and this benchmark's default are temperature 0")
    ap.add_argument("--sample-seed", type=int, default=1)
    ap.add_argument("--prefill", action="store_true", help="prompt-processing timings instead of the benchmark line")
    ap.add_argument("--prefill-batch", default="1,16")
    ap.add_argument("--prefill-len", default="512,2048")
    args = ap.parse_args()
    cfg = dict(synth.CONFIGS[args.workload])
    if args.layers:
        cfg = synth.with_layers(cfg, args.layers)
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    if args.sweep:
        run_sweep(args, cfg)
        return
    if args.prefill:
        run_prefill(args, cfg)
        return
    if args.warmup < 3:
        args.warmup = 3

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    device = f"cuda:{local_rank}"
    torch.cuda.set_device(device)
    from paper_2403_09919_b200 import binding

    B, BW, L = cfg["max_batch"], cfg["beam_width"], cfg["beam_length"]
    need = args.warmup + args.steps
    cfg["max_ctx"] = max(cfg["max_ctx"], (cfg["prompt_len"] if isinstance(cfg["prompt_len"], int) else cfg["prompt_len"][1])
                         + need * (L + 1) + 2 + BW * L)
    w = synth.make_weights(cfg, device)
    eng = binding.ReDrafter(cfg, w, device=device)
    if args.temperature > 0:
        eng.set_sampling(args.temperature, args.sample_seed)
    prompts = synth.make_prompts(cfg, B, seed=cfg.get("seed", 0) + shard_of_rank(rank)["prompt_seed_offset"])
    out = binding.AcceptOut(B, L, device)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()

    # ---- main leg: K steps, inputs resident in HBM, no host sync inside
    eng.prefill(prompts)
    for _ in range(args.warmup):
        eng.step(None, out)
    eng.poll()
    n_acc = torch.zeros(args.steps, B, dtype=torch.int32, device=device)
    n_rows = torch.zeros(args.steps, B, dtype=torch.int32, device=device)
    launches0 = eng.launch_count()
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()

    def one(i):
        eng.step(None, out)
        n_acc[i].copy_(out.n_accept)
        eng.last_packed_rows(n_rows[i])
    ms = timed_loop(eng, args.steps, one)
    clocks = sampler.stop()
    launches = eng.launch_count() - launches0
    barrier()
    eng.poll()
    tokens = int(n_acc.sum().item()) + args.steps * B
    ctx_end, _, _ = eng.get_state()
    ctx_mid = float(ctx_end.float().mean().item()) - 0.5 * tokens / B
    ms, tokens = reduce_over_ranks(ms, tokens, device)
    value = tokens / (ms * 1e-3)
    ms_per_step = ms / args.steps
    packed = packed_rows_summary(n_rows.cpu().numpy(), BW, L)

    # ---- e2e leg: the same steps driven the way a serving loop does, results read to the host each step
    pin_a = torch.zeros(B, dtype=torch.int32).pin_memory()
    pin_t = torch.zeros(B, L + 1, dtype=torch.int32).pin_memory()
    e2e_tokens = [0]

    ctx_host = [0]

    def one_e2e(i):
        eng.step(None, out)
        pin_a.copy_(out.n_accept, non_blocking=True)
        pin_t.copy_(out.tokens, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        e2e_tokens[0] += int(pin_a.sum()) + B
        # the loop knows what was accepted: it keeps the handle's context bound exact
        ctx_host[0] += int(pin_a.max()) + 1
        eng.set_ctx_bound(ctx_host[0])
    eng.prefill(prompts)
    for _ in range(args.warmup):
        eng.step(None, out)
    ctx_host[0] = int(eng.get_state()[0].max().item())
    eng.set_ctx_bound(ctx_host[0])
    barrier()
    ms_e2e = timed_loop(eng, args.steps, one_e2e)
    ms_e2e, e2e_tokens[0] = reduce_over_ranks(ms_e2e, e2e_tokens[0], device)
    e2e = {"value": e2e_tokens[0] / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 0,
           "d2h_bytes_per_step": int(B * (L + 2) * 4), "ms_per_step": ms_e2e / args.steps,
           "note": "redrafter_step through the C ABI; the accepted tokens are copied to pinned host memory and the stream "
                   "is synchronised every step; a step has no host-side input (state, KV cache and weights are device "
                   "resident by design; the prompt's H2D copy happens in redrafter_prefill, outside the decode loop)"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if cfg["dtype"] == "bf16" else "f32", "data": "synthetic", "config": workload_config(args, cfg),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "tokens_per_step": tokens / (args.steps * B * world), "packed_rows": packed}

    if rank == 0:
        # ---- roofline of the dominant kernel (the weight-streaming projection), timed per launch with CUDA events
        peak, peak_src = measured_peaks()
        prof_steps = min(8, args.steps)
        eng.prefill(prompts)
        for _ in range(args.warmup):
            eng.step(None, out)
        eng.profile(True)
        for _ in range(prof_steps):
            eng.step(None, out)
            gm = eng.profile_read(0)
            at = eng.profile_read(1)
            others = [eng.profile_read(c) for c in range(2, 8)]
        eng.profile(False)
        g_ms, g_bytes, g_n = gm
        achieved = g_bytes / (g_ms * 1e-3) / 1e9 if g_ms > 0 else 0.0
        sb = step_bytes(cfg, ctx_mid)
        # The per-launch event timing above serialises the launches: a projection timed alone cannot start its weight
        # stream under its predecessor the way it does in the running step.  The in-kernel timeline of one traced step
        # gives the rate in place: weight bytes / (last CTA done - last CTA past its dependency wait), summed over the
        # step's projections.
        in_step = None
        try:
            eng.trace(True)
            eng.step(None, out)
            torch.cuda.synchronize()
            tr = eng.trace_read().astype(np.int64)
            tb = eng.trace_bytes()
            tp = eng.trace_prefetched()
            eng.trace(False)
            sel = [i for i in range(len(tb)) if tb[i] > 0 and tr[i][6] > tr[i][2] > 0]
            body_ns = float(sum(int(tr[i][6] - tr[i][2]) for i in sel))
            if body_ns > 0:
                all_b, pre_b = float(sum(tb[i] for i in sel)), float(sum(tp[i] for i in sel))
                in_step = {"gbs": (all_b - pre_b) / body_ns, "launches": len(sel), "ms_per_step": body_ns * 1e-6,
                           "prefetched_fraction": pre_b / all_b,
                           "gbs_counting_prefetched_bytes": all_b / body_ns,
                           "dram_busy_fraction_of_step": body_ns * 1e-6 / ms_per_step,
                           "note": "in-kernel %globaltimer records of one traced step (not CUDA events).  Window of a projection: "
                                   "from the LAST CTA's dependency wait to the LAST CTA's end; gbs counts the weight bytes "
                                   "requested inside the window (every CTA's first ring-full of stages is requested before "
                                   "its wait and streams in under the preceding kernel: prefetched_fraction); "
                                   "gbs_counting_prefetched_bytes divides ALL weight bytes by the same windows and is an upper "
                                   "bound, not a rate; dram_busy_fraction_of_step = sum of the windows / step time"}
                in_step["frac_of_measured_peak"] = in_step["gbs"] / peak
        except Exception as e:  # measurement aid only
            in_step = {"error": str(e)}
        # DRAM traffic per launch: an ncu capture of six consecutive projection launches of this workload (the four of a
        # layer, the LM head and a drafter layer; summary under profiles/) read and wrote 1.040 x their algorithmic
        # bytes in total (the surplus is the activation operand and the partial sums; 1.026 in an earlier capture of
        # six other launches); traffic grows with the weight bytes, so that ratio scales the mean launch.
        NCU_TRAFFIC_RATIO = 1.040
        traffic = NCU_TRAFFIC_RATIO * g_bytes / g_n if g_n else None
        line["roofline"] = {"bound": "hbm", "kernel": "projection (weight-streaming GEMM)", "achieved": achieved, "peak": peak,
                            "unit": "GB/s", "frac": achieved / peak, "traffic": traffic,
                            "traffic_note": "bytes per launch: mean algorithmic bytes x 1.040, the DRAM read+write / algorithmic ratio of an ncu capture of six launches",
                            "algorithmic_bytes_per_launch": g_bytes / g_n if g_n else None, "peak_source": peak_src,
                            "in_step": in_step,
                            "launches_per_step": g_n / prof_steps, "ms_per_step_in_kernel": g_ms / prof_steps,
                            "attention_ms_per_step": at[0] / prof_steps,
                            "other_ms_per_step": {n: round(o[0] / prof_steps, 4) for n, o in
                                                  zip(("rmsnorm", "rope", "swiglu", "draft_select", "pack_accept", "misc"), others)},
                            "other_launches_per_step": {n: o[2] / prof_steps for n, o in
                                                        zip(("rmsnorm", "rope", "swiglu", "draft_select", "pack_accept", "misc"), others)}}
        line["headline"] = {"ms_per_step": ms_per_step, "frac_of_nominal_8tbs": sb["total"] / (ms_per_step * 1e-3) / 8e12,
                            "frac_of_measured_peak": sb["total"] / (ms_per_step * 1e-3) / 1e9 / peak,
                            "target": "north_star: >= 0.70 of the step's bytes / 8 TB/s",
                            "note": "whole step (weights + KV bytes once) against the HBM roofline; roofline.frac is the "
                                    "projection kernel timed launch by launch (serialised), roofline.in_step the same kernel in place"}
        line["bf16_logits_tolerance"] = {
            "stated": 3e-2, "met": "two-layer copies of every workload, against the unrounded and the bf16-storage oracle",
            "full_depth": "not met against the unrounded oracle and not meetable: the oracle's own bf16-storage mode is 0.040 "
                          "(7B, 32 layers), 0.057 (13B, 40) and 0.088 (33B, 60) relative L2 from its unrounded mode; the GPU "
                          "measures 0.0395 / 0.0569 / 0.0872 and is held to 1.15 x the oracle pair's distance (tests/helpers.py)"}
        line["step_roofline"] = {"algorithmic_bytes_per_step": sb["total"], "achieved_gbs": sb["total"] / (ms_per_step * 1e-3) / 1e9,
                                 "frac_of_measured_peak": sb["total"] / (ms_per_step * 1e-3) / 1e9 / peak,
                                 "frac_of_nominal_8tbs": sb["total"] / (ms_per_step * 1e-3) / 8e12,
                                 "mean_ctx": ctx_mid, "bytes": sb}
        if not args.no_extras:
            # ---- autoregressive comparator built from the same kernels, and the planted-beam mode
            n_ar = need * (L + 1) + 1
            eng.prefill(prompts)
            tok = torch.zeros(B, dtype=torch.int32, device=device)
            _, root, _ = eng.get_state()
            cont = torch.zeros(n_ar + 1, B, dtype=torch.int32, device=device)
            cont[0].copy_(root)
            for _ in range(args.warmup):
                eng.ar_step(tok)
            eng.prefill(prompts)

            def one_ar(i):
                eng.ar_step(tok)
                cont[i + 1].copy_(tok)
            ms_ar = timed_loop(eng, n_ar, one_ar)
            eng.poll()
            line["autoregressive"] = {"tokens_per_s": n_ar * B / (ms_ar * 1e-3), "ms_per_step": ms_ar / n_ar,
                                      "frac_of_measured_peak": sb["ar"] / (ms_ar / n_ar * 1e-3) / 1e9 / peak}
            cont_h = cont.cpu().numpy()                                   # [n_ar+1, B]; row 0 = root after prefill
            # Planted-beam mode, teacher-forced on the autoregressive stream: beams for every stream position are
            # planted up front; each step the host reads the accepted length (as a serving loop does), advances
            # the position and hands the step the stream's own token as root.  Accepted tokens are stream tokens by
            # construction; only a bonus token can differ (a near-tie between the two kernels' summation orders),
            # which the root hand-off overrides -- counted as "bonus_flips".
            sys.path.insert(0, os.path.join(ROOT, "tests"))
            from helpers import first_mismatch            # closed form of greedy acceptance on planted beams (test arithmetic)
            rng = np.random.default_rng(2000 + cfg.get("seed", 0))
            n_pos = n_ar - L
            table = np.zeros((n_pos, B, BW, L), dtype=np.int32)
            for p_ in range(1, n_pos):
                for b in range(B):
                    table[p_, b] = synth.plant_beams(cont_h[p_:p_ + L, b], BW, L, cfg["vocab"], rng, p=cfg.get("plant_p", 0.3),
                                                     rho=cfg.get("plant_rho", 0.0))
            table_d = torch.from_numpy(table).to(device)
            eng.prefill(prompts)
            posn = np.ones(B, dtype=np.int64)
            beams_d = torch.zeros(B, BW, L, dtype=torch.int32, device=device)
            pin_a2 = torch.zeros(B, dtype=torch.int32).pin_memory()
            pin_t2 = torch.zeros(B, L + 1, dtype=torch.int32).pin_memory()
            stats = dict(tokens=0, flips=0, closed=0, steps=0)
            rows_p = torch.zeros(args.warmup + args.steps + 1, B, dtype=torch.int32, device=device)
            step_no = [0]
            ctx_p = eng.get_state()[0].cpu().numpy().astype(np.int64)

            def one_p(i, count=True):
                for b in range(B):
                    beams_d[b].copy_(table_d[posn[b], b])
                eng.step(beams_d, out)
                pin_a2.copy_(out.n_accept, non_blocking=True)
                pin_t2.copy_(out.tokens, non_blocking=True)
                if count:
                    eng.last_packed_rows(rows_p[step_no[0]])
                    step_no[0] += 1
                torch.cuda.current_stream().synchronize()
                for b in range(B):
                    a_ = int(pin_a2[b])
                    ctx_p[b] += a_ + 1
                    if count:
                        stats["tokens"] += a_ + 1
                        stats["steps"] += 1
                        stats["closed"] += int(a_ == first_mismatch(table[posn[b], b], cont_h[posn[b]:posn[b] + L, b]).max())
                        stats["flips"] += int(int(pin_t2[b, a_]) != int(cont_h[posn[b] + a_, b]))
                    posn[b] += a_ + 1
                eng.set_state(None, cont[posn[0] - 1] if B == 1 else torch.stack([cont[posn[b] - 1, b] for b in range(B)]), None)
                eng.set_ctx_bound(int(ctx_p.max()))
            for s_ in range(args.warmup):
                one_p(s_, count=False)
            ms_p = timed_loop(eng, args.steps, one_p)
            eng.poll()
            tok_p = stats["tokens"]
            line["planted"] = {"tokens_per_s": tok_p / (ms_p * 1e-3), "ms_per_step": ms_p / args.steps,
                               "tokens_per_step": tok_p / max(1, stats["steps"]),
                               "steps_matching_closed_form": stats["closed"], "bonus_flips": stats["flips"],
                               "packed_rows": packed_rows_summary(rows_p[:step_no[0]].cpu().numpy(), BW, L),
                               "speedup_vs_autoregressive": (tok_p / ms_p) / (n_ar * B / ms_ar),
                               "note": "beams = the autoregressive stream's continuation with each token replaced at p=0.3; "
                                       "teacher-forced root, accepted length read by the host every step (one sync per step)"}
            line["speedup_vs_autoregressive"] = value / world / (n_ar * B / (ms_ar * 1e-3))
        if not args.no_cpu_baseline and world == 1:
            leg = oracle_leg(args, cfg)
            r = leg.run(args.cpu_steps, warmup=1)
            line["cpu_baseline"] = {"value": r["value"], "unit": UNIT, "cores": cpu_cores(), "kind": "oracle",
                                    "extrapolated": leg.extrapolated, "sample": r["sample"]}
            if not leg.extrapolated:
                line["cpu_baseline"]["ms_per_step"] = r["ms_per_step"]
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

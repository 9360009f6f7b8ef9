#!/usr/bin/env python
"""Benchmark of the compression pass (score + select + compact) on synthetic long-context keys.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload c3|c1|c2|c4|c0] [--mode aliased|paper] [--layers L]

One step = one fused compactor_compress call over the whole workload (every layer, KV head and
sequence).  Prints ONE JSON line.  For N > 1 (launched by torch.distributed.run, one rank per
GPU) every rank compresses its own copy of the workload (different seed): units are independent,
so there is no data-path collective and scaling is weak.
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

METRIC = "compressed tokens/s per B200 (score+select+compact)"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of the dominant kernels per head-token, from ncu captures of a smaller case of
# the same kernels (see profiles/); bytes read + written per token of one (layer, head).
# keyed by (workload, kernel); only a capture of that workload at its own retention ratio counts
NCU_TRAFFIC_BYTES_PER_HEAD_TOKEN = {("c3", "gram"): 257.1, ("c3", "score"): 260.7, ("c3", "compact"): 316.1}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--mode", default="aliased", choices=["aliased", "paper"],
                    help="aliased: score and gather the rotated keys; paper: score pre-rotation keys")
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (debugging)")
    ap.add_argument("--heads", type=int, default=None, help="override the KV-head count (slices of a few units for profiling)")
    ap.add_argument("--flush-l2", action="store_true", help="write a 256 MiB buffer before every timed step (small slices)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-units", type=int, default=None,
                    help="units in the CPU-baseline sample (default 16; 4 per step for --impl reference)")
    ap.add_argument("--no-extra", action="store_true", help="skip the other workloads, the attention term and the NLL pass")
    ap.add_argument("--fig1-n", type=int, default=None, help="with --fig1: only this context length")
    ap.add_argument("--nll", action="store_true",
                    help="time the NLL reduction of Section 3.5 on 8192 x 128256 bf16 logits instead of the headline")
    ap.add_argument("--fig1", action="store_true",
                    help="context-length sweep of the paper's Fig. 1 setting (one layer, 8 KV heads, batch 1)")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def algorithmic_bytes(w, keep, mode):
    """Bytes the method must move per step: scored K read once, kept V rows read, kept K rows
    read (a re-touch in aliased mode, so not counted there), kept K/V rows written."""
    row = w.d * 2
    per_lh = 0
    for n, kk in zip(w.seqlens, keep):
        per_lh += n * row + kk * row * (3 if mode == "aliased" else 4)
    return per_lh * w.layers * w.heads


def stage_bytes(w, keep, mode):
    """Minimal bytes of each kernel run on its own (per step)."""
    row = w.d * 2
    lh = w.layers * w.heads
    tok = sum(w.seqlens); kept = sum(keep)
    return {
        "gram": lh * tok * row,                 # the keys once (the few fp64 partial sums are not credited)
        "factor": 0,
        "score": lh * tok * (row + 4),
        "blend": 0,
        "select": lh * (tok * 4 + kept * 4),
        "compact": lh * kept * (4 * row + 4),
    }


def run_reference(args):
    """The oracle, as it stands, on the host cores: a bounded sample of the workload's units per step
    (--cpu-units, default 4: about half a second per step at the headline workload)."""
    if args.cpu_units is None:
        args.cpu_units = 4
    import numpy as np
    import torch
    from paper_2507_08143_b200 import inputs
    from oracle import compactor_oracle as orc
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = inputs.workload(args.workload, layers=args.layers)
    phi = inputs.make_sketch_matrix(w.d, w.m, w.seed).numpy()
    keep = [orc.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    sample = max(1, args.cpu_units)
    units = [(0, h % w.heads, b % w.batch) for h, b in zip(range(sample), range(sample))]
    data = []
    for (l, h, b) in units:
        kp, kr, v = inputs.make_unit(w, b, l, h)
        ks = kp if args.mode == "paper" else kr
        data.append((ks.view(torch.int16).numpy(), kr.view(torch.int16).numpy(), v.view(torch.int16).numpy(), keep[b],
                     w.seqlens[b]))

    def step():
        for ks, kr, v, kk, n in data:
            orc.compress_unit(ks, kr, v, phi, kk)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    head_tokens = sum(d[4] for d in data)
    # a token counts once for all layers x heads: scale the sample to the whole workload
    value = (head_tokens / dt) / (w.layers * w.heads)
    cores = torch.get_num_threads()
    desc = f"{len(data)} units of {w.name} per step ({head_tokens} head-tokens), scaled to {w.layers}x{w.heads} units per token"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "mode": args.mode, "layers": w.layers, "kv_heads": w.heads, "d": w.d,
                   "m": w.m, "seqlens": w.seqlens if w.batch <= 4 else f"{w.batch} sequences"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline(args, w, keep, phi):
    import torch
    if args.cpu_units is None:
        args.cpu_units = 16
    from paper_2507_08143_b200 import inputs
    from oracle import compactor_oracle as orc
    sample = max(1, args.cpu_units)
    data = []
    for i in range(sample):
        b, h = i % w.batch, i % w.heads
        kp, kr, v = inputs.make_unit(w, b, 0, h)
        ks = kp if args.mode == "paper" else kr
        data.append((ks.view(torch.int16).numpy(), kr.view(torch.int16).numpy(), v.view(torch.int16).numpy(), keep[b],
                     w.seqlens[b]))
    phi_np = phi.numpy()
    t0 = time.perf_counter()
    head_tokens, passes = 0, 0
    while time.perf_counter() - t0 < 12.0:                 # about 12 s of CPU work
        for ks, kr, v, kk, n in data:
            orc.compress_unit(ks, kr, v, phi_np, kk)
            head_tokens += n
        passes += 1
    dt = time.perf_counter() - t0
    value = (head_tokens / dt) / (w.layers * w.heads)
    return {"value": value, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
            "sample": f"{sample} distinct units of {w.name} x {passes} passes ({head_tokens} head-tokens, {dt:.1f} s), "
                      f"scaled to {w.layers}x{w.heads} units per token"}


# The paper's Fig. 1 (one layer of Llama-3.1-8B, batch 1, NVIDIA H100 80GB, median wall-clock ms) for the
# leverage-score-only curve, as context beside our numbers for the same shape.
FIG1_PAPER_FULL_MS_H100 = {256: 1.026687, 512: 1.032664, 1024: 1.046611, 2048: 1.081453, 4096: 1.145309,
                           8192: 1.274366, 16384: 1.518961, 32768: 2.001249, 65536: 2.975803, 131072: 5.902795,
                           262144: 7.768950, 524288: 19.506534, 1048576: 31.583626}
FIG1_PAPER_MS_H100 = {256: 1.345554, 512: 1.312034, 1024: 1.287826, 2048: 1.276906, 4096: 1.274009,
                      8192: 1.276523, 16384: 1.301756, 32768: 1.428951, 65536: 1.588616, 131072: 1.924723,
                      262144: 2.654723, 524288: 4.030933, 1048576: 6.812491}


def run_fig1(args):
    """Median time of compactor_score, and of the whole compactor_compress at 30 % retention, on
    8 KV heads x n tokens, for the context lengths of the paper's Fig. 1."""
    import torch
    from paper_2507_08143_b200 import binding as B, inputs
    torch.cuda.set_device(0)
    rows = []
    for n in sorted(FIG1_PAPER_MS_H100):
        if args.fig1_n is not None and n != args.fig1_n:
            continue
        w = inputs.Workload(f"fig1-n{n}", 1, 8, 128, [n], [0.3], p=0.7, n_out=4, theta=5e5, seed=100)
        _, kr, v = inputs.make_tensors(w, device="cuda", want_pre=False)
        shape = B.Shape(1, 8, 128, 48, [n])
        keep = [B.keep_count(n, 0.3)]
        phi = inputs.make_sketch_matrix(128, 48, 0).cuda()
        scores = torch.empty(1, 8, n, dtype=torch.float32, device="cuda")
        idx = torch.empty(1, 8, keep[0], dtype=torch.int32, device="cuda")
        ko = torch.empty(1, 8, keep[0], 128, dtype=torch.bfloat16, device="cuda"); vo = torch.empty_like(ko)
        ws = B.alloc_workspace(shape)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # larger than L2

        def timed(fn, iters):
            out = []
            for _ in range(3):
                fn()
            for _ in range(iters):
                flush.zero_()                                                  # start every call L2-cold
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); fn(); e1.record(); torch.cuda.synchronize()
                out.append(e0.elapsed_time(e1))
            return statistics.median(out)

        iters = max(5, args.steps)
        t_score = timed(lambda: B.score(shape, kr, phi, scores, ws), iters)
        t_full = timed(lambda: B.compress(shape, kr, kr, v, phi, keep, idx, ko, vo, ws, scores_out=scores), iters)
        # the same call recorded into a CUDA graph once and replayed: one launch instead of seven
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            B.compress(shape, kr, kr, v, phi, keep, idx, ko, vo, ws, scores_out=scores)
        t_graph = timed(graph.replay, iters)
        del graph
        # the paper's full score: attention term of the 4 query heads per KV head (Llama-3.1-8B), blended
        q = inputs.make_queries(w, 4, device="cuda")
        attn = torch.empty(1, 8, n, dtype=torch.float32, device="cuda")

        def full_score():
            B.attention_scores(shape, q, kr, 4, attn, ws, scale=128 ** -0.5, pool=7)
            B.score(shape, kr, phi, scores, ws, attn=attn, lam=0.3)

        t_attn = timed(lambda: B.attention_scores(shape, q, kr, 4, attn, ws, scale=128 ** -0.5, pool=7), iters)
        t_both = timed(full_score, iters)
        rows.append({"n": n, "score_ms": round(t_score, 4), "compress_ms": round(t_full, 4),
                     "compress_graph_ms": round(t_graph, 4),
                     "attention_ms": round(t_attn, 4), "full_score_ms": round(t_both, 4),
                     "paper_h100_score_ms": FIG1_PAPER_MS_H100[n], "paper_h100_full_ms": FIG1_PAPER_FULL_MS_H100[n]})
        del kr, v, scores, idx, ko, vo, ws, flush, q, attn
        torch.cuda.empty_cache()
    print(json.dumps({"fig1": rows, "shape": "1 layer x 8 KV heads (x 4 query heads for the attention term), d=128, m=48, "
                                             "batch 1, bf16, keep 30 %",
                      "timing": "median of CUDA-event times, L2 flushed before every call"}))


def run_nll(args):
    """Streaming rate of compactor_nll on synthetic logits of a 128K-entry vocabulary."""
    import torch
    from paper_2507_08143_b200 import binding as B
    torch.cuda.set_device(0)
    rows, vocab = 8192, 128256
    g = torch.Generator(device="cuda"); g.manual_seed(7)
    logits = (torch.randn(rows, vocab, device="cuda", generator=g) * 4).to(torch.bfloat16)
    targets = torch.randint(0, vocab, (rows,), device="cuda", generator=g, dtype=torch.int32)
    row_nll = torch.empty(rows, dtype=torch.float32, device="cuda")
    out = torch.empty(1, dtype=torch.float64, device="cuda")
    for _ in range(max(3, args.warmup)):
        B.nll(logits, targets, [rows], row_nll, out)
    times = []
    for _ in range(max(5, args.steps)):                     # 2.1 GB of logits per call: larger than L2
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); B.nll(logits, targets, [rows], row_nll, out); e1.record(); torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    ms = statistics.median(times)
    peak, kind = measured_peak()
    gbs = rows * vocab * 2 / ms / 1e6
    print(json.dumps({"nll": {"rows": rows, "vocab": vocab, "dtype": "bf16", "ms": round(ms, 4), "GB/s": round(gbs, 1),
                              "frac": round(gbs / peak, 4), "peak": peak, "peak_kind": "of " + kind,
                              "mean_nll": float(out.cpu()[0])}}))


def time_workload(B, inputs, torch, name, mode, steps, warmup):
    """One workload through the fused call: ms per step, stage times, fraction of the HBM roofline."""
    w = inputs.workload(name)
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    phi_d = inputs.make_sketch_matrix(w.d, w.m, w.seed).cuda()
    kp, kr, v = inputs.make_tensors(w, device="cuda", want_pre=(mode == "paper"))
    k_score = kp if mode == "paper" else kr
    total_keep = sum(keep)
    idx = torch.empty(w.layers, w.heads, total_keep, dtype=torch.int32, device="cuda")
    k_out = torch.empty(w.layers, w.heads, total_keep, w.d, dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)
    status = torch.zeros(w.units, dtype=torch.int32, device="cuda")
    ws = B.alloc_workspace(shape)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")           # larger than L2
    small = w.layers * w.heads * w.total_tokens * w.d * 2 < (512 << 20)          # inputs near the L2 size: flush between steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(B.N_STAGE_EVENTS)] for _ in range(steps)]
    for es in ev:
        for e in es:
            e.record()
    for _ in range(max(warmup, 3)):
        B.compress(shape, k_score, kr, v, phi_d, keep, idx, k_out, v_out, ws, status=status)
    torch.cuda.synchronize()
    pairs = []                                            # the step itself: the plain call, nothing between its kernels,
    for _ in range(steps):                                # steps enqueued back to back (the flush is outside the events)
        if small:
            flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.compress(shape, k_score, kr, v, phi_d, keep, idx, k_out, v_out, ws, status=status)
        e1.record()
        pairs.append((e0, e1))
    torch.cuda.synchronize()
    ms = statistics.median(a.elapsed_time(b) for a, b in pairs)
    for es in ev:                                         # stage times: the same call with markers between its kernels
        if small:
            flush.zero_()
        B.compress_profiled(shape, k_score, kr, v, phi_d, keep, idx, k_out, v_out, ws, es, status=status)
    torch.cuda.synchronize()
    assert int(status.max().item()) == 0
    stage_ms = {nm: statistics.median(es[j].elapsed_time(es[j + 1]) for es in ev) for j, nm in enumerate(B.STAGE_NAMES)}
    peak, _ = measured_peak()
    b_alg = algorithmic_bytes(w, keep, mode)
    gbs = b_alg / (ms * 1e-3) / 1e9
    del kp, kr, v, idx, k_out, v_out, ws, flush
    torch.cuda.empty_cache()
    return {"workload": w.name, "mode": mode, "units": w.units, "tokens": w.total_tokens, "ms_per_step": round(ms, 4),
            "tokens_per_s": round(w.total_tokens / (ms * 1e-3)), "stage_ms": {k: round(t, 4) for k, t in stage_ms.items()},
            "path_roofline": {"algorithmic_bytes_per_step": b_alg, "achieved": round(gbs, 1), "frac": round(gbs / peak, 4)},
            "l2": "flushed before every step" if small else "inputs exceed L2"}


def time_full_variant(B, inputs, torch, name, selection, factorization, steps, warmup):
    """A workload through compactor_compress_full without the attention term: selection across the heads of a
    layer, or the eigendecomposition route of the scorer, at full size."""
    w = inputs.workload(name)
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    phi_d = inputs.make_sketch_matrix(w.d, w.m, w.seed).cuda()
    _, kr, v = inputs.make_tensors(w, device="cuda", want_pre=False)
    total_keep = sum(keep)
    idx = torch.empty(w.layers, w.heads * total_keep, dtype=torch.int32, device="cuda")
    offs = torch.empty(w.layers, w.batch, w.heads + 1, dtype=torch.int32, device="cuda")
    k_out = torch.empty(w.layers, w.heads * total_keep, w.d, dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)
    status = torch.zeros(w.units, dtype=torch.int32, device="cuda")
    opt = B.options(selection=selection, factorization=factorization, eig_floor=1e-6, lam=0.0, q_per_kv=0)
    ws = torch.empty(B.compress_full_workspace_bytes(shape, opt), dtype=torch.uint8, device="cuda")
    call = lambda: B.compress_full(shape, opt, None, kr, kr, v, phi_d, keep, idx, k_out, v_out, ws,
                                   head_offsets_out=offs, status=status)
    for _ in range(max(warmup, 3)):
        call()
    pairs = []
    for _ in range(steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); call(); e1.record()
        pairs.append((e0, e1))
    torch.cuda.synchronize()
    ms = statistics.median(a.elapsed_time(b) for a, b in pairs)
    timeouts = int((status & 4).max().item())             # 4 = a bounded wait ran out; the eigen route reports floored eigenvalues with 2
    del kr, v, idx, k_out, v_out, ws
    torch.cuda.empty_cache()
    assert timeouts == 0
    return {"workload": w.name, "units": w.units, "tokens": w.total_tokens, "ms_per_step": round(ms, 4),
            "tokens_per_s": round(w.total_tokens / (ms * 1e-3))}


def extra_measurements(args, B, inputs, torch):
    """The other benchmark workloads, the attention term, the full method and the NLL pass: a few timed
    steps each (medians of CUDA-event times), reported beside the headline."""
    out = {"other_workloads": {}}
    steps = 5
    for key, name, mode in (("c1", "c1", "aliased"), ("c2", "c2", "aliased"), ("c4", "c4", "aliased"), ("c3-paper", "c3", "paper")):
        out["other_workloads"][key] = time_workload(B, inputs, torch, name, mode, steps, 3)
    # the headline workload through the one-call entry point: selection across heads (Section 3.4), and the
    # eigendecomposition route of Appendix C with its floor
    out["other_workloads"]["c3-across-heads"] = time_full_variant(B, inputs, torch, "c3", B.SELECT_ACROSS_HEADS,
                                                                  B.FACTOR_CHOLESKY, steps, 3)
    out["other_workloads"]["c3-eig-route"] = time_full_variant(B, inputs, torch, "c3", B.SELECT_PER_HEAD, B.FACTOR_EIG, steps, 3)
    # the paper's Fig. 1 shape at n = 131072: one layer, 8 KV heads x 4 query heads, batch 1
    n, G = 131072, 4
    w = inputs.Workload("fig1-n131072", 1, 8, 128, [n], [0.3], p=0.7, n_out=4, theta=5e5, seed=100)
    _, kr, v = inputs.make_tensors(w, device="cuda", want_pre=False)
    q = inputs.make_queries(w, G, device="cuda")
    shape = B.Shape(1, 8, 128, 48, [n])
    keep = [B.keep_count(n, 0.3)]
    phi = inputs.make_sketch_matrix(128, 48, 0).cuda()
    attn = torch.empty(1, 8, n, dtype=torch.float32, device="cuda")
    ws = B.alloc_workspace(shape)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def timed(fn, iters=7):
        for _ in range(3):
            fn()
        ts = []
        for _ in range(iters):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record(); torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return statistics.median(ts)

    t_attn = timed(lambda: B.attention_scores(shape, q, kr, G, attn, ws, scale=128 ** -0.5, pool=7))
    flops = 2.0 * 8 * G * n * 256 * 128                                  # Q K^T of every 256-token chunk
    out["attention"] = {"shape": "1 layer x 8 KV heads x 4 query heads, n = 131072, chunk 256, pool 7", "ms": round(t_attn, 4),
                        "qk_tflops": round(flops / (t_attn * 1e-3) / 1e12, 1)}
    opt = B.options(selection=B.SELECT_ACROSS_HEADS, lam=0.3, q_per_kv=G, scale=128 ** -0.5, pool=7)
    idx = torch.empty(1, 8 * keep[0], dtype=torch.int32, device="cuda")
    offs = torch.empty(1, 1, 9, dtype=torch.int32, device="cuda")
    ko = torch.empty(1, 8 * keep[0], 128, dtype=torch.bfloat16, device="cuda"); vo = torch.empty_like(ko)
    wsf = torch.empty(B.compress_full_workspace_bytes(shape, opt), dtype=torch.uint8, device="cuda")
    t_full = timed(lambda: B.compress_full(shape, opt, q, kr, kr, v, phi, keep, idx, ko, vo, wsf, head_offsets_out=offs))
    out["full_method"] = {"shape": "as above, keep 30 %, lambda 0.3, m 48, selection across heads; one compactor_compress_full call",
                          "ms": round(t_full, 4),
                          "paper_h100_full_score_ms": FIG1_PAPER_FULL_MS_H100[n],
                          "note": "the paper's figure is the scoring time alone on an H100 80GB (context, not a target)"}
    del kr, v, q, attn, ws, idx, ko, vo, wsf
    torch.cuda.empty_cache()
    rows, vocab = 8192, 128256
    g = torch.Generator(device="cuda"); g.manual_seed(7)
    logits = (torch.randn(rows, vocab, device="cuda", generator=g) * 4).to(torch.bfloat16)
    targets = torch.randint(0, vocab, (rows,), device="cuda", generator=g, dtype=torch.int32)
    row_nll = torch.empty(rows, dtype=torch.float32, device="cuda")
    res = torch.empty(1, dtype=torch.float64, device="cuda")
    t_nll = timed(lambda: B.nll(logits, targets, [rows], row_nll, res))
    peak, _ = measured_peak()
    gbs = rows * vocab * 2 / t_nll / 1e6
    out["nll"] = {"rows": rows, "vocab": vocab, "dtype": "bf16", "ms": round(t_nll, 4), "GB/s": round(gbs, 1), "frac": round(gbs / peak, 4)}
    return out


def main():
    args = parse_args()
    if args.nll:
        run_nll(args)
        return
    if args.impl == "reference":
        run_reference(args)
        return
    if args.fig1:
        run_fig1(args)
        return

    import torch
    from paper_2507_08143_b200 import binding as B, inputs, sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    w = sharding.rank_workload(inputs.workload(args.workload, layers=args.layers), rank)
    if args.heads is not None:
        w.heads = args.heads
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    total_keep = sum(keep)
    phi = inputs.make_sketch_matrix(w.d, w.m, w.seed)
    phi_d = phi.cuda()

    kp, kr, v = inputs.make_tensors(w, device="cuda", want_pre=(args.mode == "paper"))
    k_score = kp if args.mode == "paper" else kr
    L, Hh = w.layers, w.heads
    idx = torch.empty(L, Hh, total_keep, dtype=torch.int32, device="cuda")
    k_out = torch.empty(L, Hh, total_keep, w.d, dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)
    status = torch.zeros(L * Hh * w.batch, dtype=torch.int32, device="cuda")
    ws = B.alloc_workspace(shape)

    events = [torch.cuda.Event(enable_timing=True) for _ in range(B.N_STAGE_EVENTS * args.steps)]
    for e in events:
        e.record()
    torch.cuda.synchronize()

    def step(ev=None):
        if ev is None:
            B.compress(shape, k_score, kr, v, phi_d, keep, idx, k_out, v_out, ws, status=status)
        else:
            B.compress_profiled(shape, k_score, kr, v, phi_d, keep, idx, k_out, v_out, ws, ev, status=status)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    t_beg, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if args.flush_l2 else None
    t_beg.record()
    for i in range(args.steps):
        if flush is not None:
            flush.zero_()
        step(events[i * B.N_STAGE_EVENTS:(i + 1) * B.N_STAGE_EVENTS])
    t_end.record()
    barrier()
    elapsed_ms = t_beg.elapsed_time(t_end)
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = sharding.max_over_ranks(elapsed_ms, dist, device="cuda")
    ms_per_step = elapsed_ms / args.steps
    value = sharding.job_tokens_per_second(w.total_tokens, world, ms_per_step)
    assert int(status.max().item()) == 0, "a unit reported a numerical status flag"

    # per-kernel times from the stage markers of the timed region
    stage_ms = {name: 0.0 for name in B.STAGE_NAMES}
    for i in range(args.steps):
        ev = events[i * B.N_STAGE_EVENTS:(i + 1) * B.N_STAGE_EVENTS]
        for j, name in enumerate(B.STAGE_NAMES):
            stage_ms[name] += ev[j].elapsed_time(ev[j + 1]) / args.steps
    sb = stage_bytes(w, keep, args.mode)
    dominant = max(stage_ms, key=stage_ms.get)
    peak, peak_kind = measured_peak()
    achieved = sb[dominant] / (stage_ms[dominant] * 1e-3) / 1e9
    traffic = NCU_TRAFFIC_BYTES_PER_HEAD_TOKEN.get((args.workload, dominant)) if args.layers is None and args.heads is None else None
    if traffic is not None:
        traffic = traffic * L * Hh * w.total_tokens
    b_alg = algorithmic_bytes(w, keep, args.mode)
    path_gbs = b_alg / (ms_per_step * 1e-3) / 1e9

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 inputs, fp32 tensor-core accumulate, fp64 factorisation",
        "data": "synthetic",
        "config": {"workload": w.name, "mode": args.mode, "layers": L, "kv_heads": Hh, "d": w.d, "m": w.m,
                   "seqlens": w.seqlens if w.batch <= 4 else f"{w.batch} sequences, {w.total_tokens} tokens",
                   "keep": keep if w.batch <= 4 else total_keep, "units_per_gpu": w.units,
                   "l2": "inputs (GBs per step) far exceed the 126 MB L2; no flush needed"},
        "head_tokens_per_s": value * L * Hh,
        "gpu_launches": 7 * args.steps,       # table upload, Gram pass, projection, Cholesky, scoring pass, selection, compaction
        "stage_ms": {k: round(t, 4) for k, t in stage_ms.items()},
        "roofline": {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_kind": f"of {peak_kind}",
                     "bytes_per_launch": sb[dominant]},
        "path_roofline": {"algorithmic_bytes_per_step": b_alg, "achieved": path_gbs, "peak": peak, "unit": "GB/s",
                          "frac": path_gbs / peak, "frac_of_8TBs": path_gbs / 8000.0},
        "clocks": clocks,
    }

    if not args.no_e2e:
        result["e2e"] = e2e(args, B, w, shape, keep, phi_d, k_score, kr, v, dist, world)
    if rank == 0 and world == 1 and not args.no_cpu:
        result["cpu_baseline"] = cpu_baseline(args, w, keep, phi)
    if rank == 0 and world == 1 and not args.no_extra:
        del kp, kr, v, k_score, idx, k_out, v_out, ws
        torch.cuda.empty_cache()
        result.update(extra_measurements(args, B, inputs, torch))
    if rank == 0:
        print(json.dumps(result))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def e2e(args, B, w, shape, keep, phi_d, k_score, kr, v, dist, world):
    """The same pass with HOST inputs and outputs: the workload is streamed in groups of layers
    through pinned host buffers (host->device copy of the group's K and V, compress, device->host
    copy of indices and compressed K/V), every step."""
    import torch
    group = max(g for g in range(1, 9) if w.layers % g == 0)      # layers per group: a divisor, at most 8
    n_groups = w.layers // group
    g_shape = B.Shape(group, w.heads, w.d, w.m, w.seqlens)
    total_keep = sum(keep)
    T = w.total_tokens
    paper = args.mode == "paper"
    # pinned host copies of one group of layers (the first), reused for every group of the step
    hk = torch.empty(group, w.heads, T, w.d, dtype=torch.bfloat16).pin_memory()
    hv = torch.empty_like(hk).pin_memory()
    hk.copy_(kr[:group]); hv.copy_(v[:group])
    hs = None
    if paper:
        hs = torch.empty_like(hk).pin_memory(); hs.copy_(k_score[:group])
    h_idx = torch.empty(group, w.heads, total_keep, dtype=torch.int32).pin_memory()
    h_ko = torch.empty(group, w.heads, total_keep, w.d, dtype=torch.bfloat16).pin_memory()
    h_vo = torch.empty_like(h_ko).pin_memory()
    dk = [torch.empty_like(hk, device="cuda") for _ in range(2)]
    dv = [torch.empty_like(hk, device="cuda") for _ in range(2)]
    ds = [torch.empty_like(hk, device="cuda") for _ in range(2)] if paper else dk
    d_idx = [torch.empty(group, w.heads, total_keep, dtype=torch.int32, device="cuda") for _ in range(2)]
    d_ko = [torch.empty(group, w.heads, total_keep, w.d, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    d_vo = [torch.empty_like(d_ko[0]) for _ in range(2)]
    ws = B.alloc_workspace(g_shape)
    copy_in, copy_out = torch.cuda.Stream(), torch.cuda.Stream()
    main = torch.cuda.current_stream()

    def one_step():
        in_done = [torch.cuda.Event() for _ in range(n_groups)]
        comp_done = [torch.cuda.Event() for _ in range(n_groups)]
        out_done = [torch.cuda.Event() for _ in range(n_groups)]
        for g in range(n_groups):
            s = g & 1
            with torch.cuda.stream(copy_in):
                if g >= 2:
                    copy_in.wait_event(comp_done[g - 2])      # slot's previous inputs consumed
                dk[s].copy_(hk, non_blocking=True); dv[s].copy_(hv, non_blocking=True)
                if paper:
                    ds[s].copy_(hs, non_blocking=True)
                in_done[g].record(copy_in)
            main.wait_event(in_done[g])
            if g >= 2:
                main.wait_event(out_done[g - 2])              # slot's previous outputs copied out
            B.compress(g_shape, ds[s], dk[s], dv[s], phi_d, keep, d_idx[s], d_ko[s], d_vo[s], ws)
            comp_done[g].record(main)
            with torch.cuda.stream(copy_out):
                copy_out.wait_event(comp_done[g])
                h_idx.copy_(d_idx[s], non_blocking=True)
                h_ko.copy_(d_ko[s], non_blocking=True); h_vo.copy_(d_vo[s], non_blocking=True)
                out_done[g].record(copy_out)
        main.wait_event(out_done[-1])

    steps = max(1, min(args.steps, 3))
    one_step()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        one_step()
    t1.record()
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / steps
    from paper_2507_08143_b200 import sharding
    ms = sharding.max_over_ranks(ms, dist, device="cuda")
    row = w.d * 2
    h2d = n_groups * group * w.heads * T * row * (3 if paper else 2)
    d2h = n_groups * group * w.heads * total_keep * (2 * row + 4)
    return {"value": w.total_tokens * world / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "how": f"{n_groups} groups of {group} layers streamed through pinned host buffers, double-buffered"}


if __name__ == "__main__":
    main()

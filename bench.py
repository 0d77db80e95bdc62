#!/usr/bin/env python
"""Benchmark of the OBCache hot path (score -> pool/select -> compact) on B200.

A "step" is one pass of the whole path over one Llama-3-8B-shaped layer cache (32 query heads /
8 KV heads, head_dim 128, N = 32768 cached tokens, window W = 32, bf16, OBCache-V&K, max-pool 7,
budget 2048 per head).  The metric is cached tokens scored+compacted per second per layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

With N > 1 it is launched by torch.distributed.run, one rank per GPU; every rank processes its
own cache (the (batch, KV head) units are independent, so there is no data-path collective) and
the reported value is the sum over ranks divided by the slowest rank's time (weak scaling).

Timing: W warm-up steps, then rounds of exactly K steps, each round bracketed by a barrier and a
device synchronisation and timed with CUDA events; rounds are repeated until at least half a
second has been timed and the median round is reported (with few steps a single round lasts a
millisecond or two, less than one clock sample).  Every workload prints one JSON line with the
clocks sampled during the rounds, the roofline of its dominant kernel and of the whole step, the
plain-ALU and special-function bounds, and the CPU checker timed on a bounded sample.

`--impl reference` times the CPU checker (oracle/) as it stands on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "cached tokens scored+compacted/sec per layer"
UNIT = "tokens/s"
WORKLOAD = ("llama3-8b-layer-32k: B1 Hq32 Hkv8 d128 N32768 W32 bf16, OBCache-V&K, max-pool 7, "
            "budget 2048/head, n_recent 32")
NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 8000.0, 2250.0
N_SM, FP32_LANES, SFU_LANES = 148, 128, 16        # per SM: fp32 lanes, special-function lanes
MIN_TIMED_S = 0.5
PREFILL = {"llama32k": 2, "qwen128k": 3, "ragged": 4}
WORKLOADS = ["llama32k", "qwen128k", "ragged", "decode", "llama32k-given", "qwen128k-given", "llama32k-adaptive",
             "history4k", "decode-window", "llama32k-sharded"]


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    sm_max_mhz=float(d.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, sm_max_mhz=1965.0,
                source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons in the background."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.t0 = time.time()
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu=timestamp,{self.FIELDS}", "--format=csv,noheader,nounits",
                                       "-lms", "20", "-i", str(device_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None
        self.marks = {}

    def mark(self, name):
        self.marks[name] = time.time()

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.05)
        self.p.terminate()
        self.p.wait()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        from datetime import datetime
        parsed = []
        for r in rows:
            try:
                ts = datetime.strptime(r[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                parsed.append((ts, float(r[1]), float(r[2]), float(r[3]), r[4:8]))
            except (ValueError, IndexError):
                continue
        a, b = self.marks.get("timed_begin", self.t0), self.marks.get("timed_end", time.time())
        inside = [x for x in parsed if a <= x[0] <= b]
        where = "timed rounds"
        if not inside:                       # region shorter than the sampling period
            inside, where = parsed, "whole run"
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for x in inside for n, v in zip(names, x[4]) if v.strip() == "Active"})
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(x[1] for x in inside), "sm_max_mhz": inside[0][2],
                "power_w_max": max(x[3] for x in inside), "reasons": reasons, "samples": len(inside),
                "window": where}


def ncu_traffic(workload, kernel):
    """DRAM bytes per launch of `kernel` on `workload` from the committed ncu summaries, or None when there is
    no capture for that pair or the kernel's source file has changed since it was taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "traffic.txt")
    if not os.path.exists(path):
        return None
    rec = dict(l.split() for l in open(path) if l.strip() and not l.startswith("#"))
    key = f"{workload}.{kernel}"
    if key not in rec:
        return None
    source = "decode.cu" if kernel.startswith("decode") else "score_tc.cu"
    src = os.path.join(ROOT, "paper_2510_07651_b200", "csrc", source)
    if rec.get("sha256." + source) != hashlib.sha256(open(src, "rb").read()).hexdigest():
        return None
    return float(rec[key])


# ---------------------------------------------------------------------------------------------------
# what each workload is: name, how the inputs relate to the L2, how it shards
# ---------------------------------------------------------------------------------------------------
def workload_config(name, world=1):
    """The `config` object of the JSON line: the same for the library arm and the reference arm."""
    text = {
        "llama32k": WORKLOAD,
        "qwen128k": "qwen2.5-7b-layer-128k: B1 Hq28 Hkv4 d128 N131072 W64 bf16, OBCache-K and V&K (one launch), max-pool 7, "
                    "budget 4096/head, n_recent 64",
        "ragged": "llama3-8b-layer, batch 8, ragged lengths uniform in [8192, 65536] (seeded): Hq32 Hkv8 d128 W32 bf16, "
                  "OBCache-V&K, no pooling, budget 10% of each length, n_recent 32",
        "decode": "decode rescoring: B32 Hq32 Hkv8 d128 bf16, live 4096 -> 4097 -> 4096 slots per head and step (a 16384-token "
                  "context already reduced to the 4096 budget), W1, OBCache-V&K accumulated, 4 sinks, 256 recent, one eviction "
                  "per head per step",
        "decode-window": "decode rescoring as `decode`, the accumulator limited to the scores of the last 16 steps",
        "llama32k-given": WORKLOAD + "; window O and LSE supplied by the caller (no attention recompute)",
        "qwen128k-given": "qwen2.5-7b-layer-128k as `qwen128k`; window O and LSE supplied by the caller (no attention recompute)",
        "llama32k-adaptive": WORKLOAD + "; head-adaptive budgets (safeguard 0.2) instead of one budget per head",
        "history4k": "llama3-8b-layer, whole sequence as perturbation window: B1 Hq32 Hkv8 d128 N4096 W4096 bf16 (16384 window "
                     "rows per KV head, causal), OBCache-V&K, max-pool 7, budget 512/head",
        "llama32k-sharded": "one of two ranks of the 32k Llama layer sharded by token range (this rank: tokens 16384..32767), "
                            "emulated on one GPU: window attention of the shard, merge with the peer's (o, lse), local scores, "
                            "selection over the gathered scores; no compaction",
    }[name]
    l2 = {
        "llama32k": "4 distinct input copies rotated between steps (4 x 135 MB > 126 MB L2)",
        "llama32k-given": "4 distinct input copies rotated between steps (4 x 135 MB > 126 MB L2)",
        "llama32k-adaptive": "4 distinct input copies rotated between steps (4 x 135 MB > 126 MB L2)",
        "qwen128k": "inputs larger than L2 (K+V = 268 MB)", "qwen128k-given": "inputs larger than L2 (K+V = 268 MB)",
        "ragged": "inputs larger than L2 (K+V = 1.2 GB)",
        "decode": "inputs larger than L2 (live K+V = 537 MB per step)",
        "decode-window": "inputs larger than L2 (live K+V = 537 MB per step)",
        "history4k": "16 distinct input copies rotated between steps (16 x 17 MB > 2 x 126 MB L2)",
        "llama32k-sharded": "4 distinct input copies rotated between steps (4 x 67 MB > 2 x 126 MB L2)",
    }[name]
    return {"workload": text, "l2": l2,
            "parallelism": f"{world} independent layer caches, one per GPU, no collective"}


def time_rounds(run_step, steps, warmup, barrier, min_total_s=None, max_rounds=2000):
    """Median over rounds of exactly `steps` steps; each round has a barrier + synchronise on both sides.
    Returns (median ms per round, number of rounds)."""
    import torch
    from paper_2510_07651_b200 import multirank
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    min_total_s = MIN_TIMED_S if min_total_s is None else min_total_s
    for i in range(warmup):
        run_step(i)
    rounds, total, it = [], 0.0, warmup
    while True:
        barrier()
        e0.record()
        for _ in range(steps):
            run_step(it); it += 1
        e1.record()
        torch.cuda.synchronize()
        barrier()
        ms = multirank.max_over_ranks(e0.elapsed_time(e1), "cuda")      # every rank sees the same figure
        rounds.append(ms); total += ms * 1e-3
        if total >= min_total_s or len(rounds) >= max_rounds:
            break
    time_rounds.last = {"first_round_ms": rounds[0], "fastest_round_ms": min(rounds), "slowest_round_ms": max(rounds)}
    return statistics.median(rounds), len(rounds)


def bounds_of(alg, seconds, peaks, clock_mhz):
    """Roofline record of one kernel (or of the whole step) from its algorithmic work.
    alg: dict(bytes, flops, pairs, fp32_per_pair, ex2_per_pair)."""
    t_hbm = alg["bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_mma = alg.get("flops", 0) / (peaks["bf16_tflops_sustained"] * 1e12)
    rec = {"algorithmic_bytes": alg["bytes"], "algorithmic_flops": alg.get("flops", 0),
           "t_hbm_us": t_hbm * 1e6, "t_mma_us": t_mma * 1e6}
    if t_hbm >= t_mma:
        ach = alg["bytes"] / seconds / 1e9
        rec.update(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"],
                   frac_of_nominal=ach / NOMINAL_HBM_GBS, nominal_peak=NOMINAL_HBM_GBS,
                   peak_source=f"{peaks['source']} STREAM-style copy")
    else:
        ach = alg["flops"] / seconds / 1e12
        rec.update(bound="tensor", achieved=ach, peak=peaks["bf16_tflops_sustained"], unit="TFLOP/s",
                   frac=ach / peaks["bf16_tflops_sustained"], frac_of_nominal=ach / NOMINAL_BF16_TFLOPS,
                   nominal_peak=NOMINAL_BF16_TFLOPS, peak_source=f"{peaks['source']} cuBLAS bf16 sustained")
    if alg.get("pairs"):
        hz = (clock_mhz or peaks["sm_max_mhz"]) * 1e6
        rec["t_fp32_us"] = alg["pairs"] * alg["fp32_per_pair"] / (N_SM * FP32_LANES * hz) * 1e6
        rec["t_sfu_us"] = alg["pairs"] * alg["ex2_per_pair"] / (N_SM * SFU_LANES * hz) * 1e6
        rec["alu_note"] = (f"{alg['pairs']:.3g} (row, token) pairs x {alg['fp32_per_pair']} fp32 instructions on {N_SM} x {FP32_LANES} "
                           f"lanes and x {alg['ex2_per_pair']} ex2 on {N_SM} x {SFU_LANES} lanes at {hz / 1e6:.0f} MHz")
    return rec


def prefill_model(case, run, given=False):
    """Algorithmic work of the prefill path on `case`: per kernel kind and for the whole step."""
    d, es = case.d, 2 if case.dtype == "bf16" else 4
    tok_heads = int(case.seq_lens.sum()) * case.Hkv                  # cached tokens x KV heads
    planes = len(run["variants"])
    # (row, token) pairs a pass visits: every window row sees the tokens up to its own position
    pairs = 0
    for n in case.seq_lens:
        n = int(n)
        vis = sum(n - case.W + i + 1 for i in range(case.W)) if case.W < 4096 else case.W * (2 * n - case.W + 1) // 2
        pairs += vis * case.G * case.Hkv
    kv = tok_heads * d * es * 2
    contraction = 2 * d * pairs                                      # flops of one contraction over the visible pairs
    fp32 = 7 if run["variants"] == ["VK"] else 10 if set(run["variants"]) == {"K", "VK"} else 12
    budgets = run["budget"] if isinstance(run["budget"], list) else [run["budget"]] * case.B
    kept = sum(min(int(b), int(n)) for b, n in zip(budgets, case.seq_lens)) * case.Hkv
    gather = kept * d * es * 2 * 2                                   # K and V rows read and written
    score_rw = tok_heads * 4 * (planes + 1)                          # planes written, the selected plane read
    model = {
        "pass1": dict(bytes=kv, flops=2 * contraction, pairs=pairs, fp32_per_pair=5, ex2_per_pair=1),
        "pass2": dict(bytes=kv + tok_heads * 4 * planes, flops=2 * contraction, pairs=pairs, fp32_per_pair=fp32, ex2_per_pair=1),
        "gather": dict(bytes=gather), "select": dict(bytes=tok_heads * 4 + kept * 4),
        "step": dict(bytes=kv + score_rw + gather + kept * 4, flops=(2 if given else 4) * contraction,
                     pairs=pairs * (1 if given else 2), fp32_per_pair=(fp32 if given else (fp32 + 5) / 2), ex2_per_pair=1),
    }
    return model


def kernel_kind(name):
    for k in ("pass1", "pass2", "gather", "select"):
        if k in name:
            return k
    return None


def finish_line(*, name, world, args, metric, unit, value, ms_round, rounds, prof, prof_steps, model, peaks, clocks,
                cpu, e2e=None, headline_kernel=None, spans=None, extra=None, launch=None, timing_detail=None):
    ms_step = ms_round / args.steps
    clock = clocks.get("sm_mhz") if clocks else None
    kernels = {k: {"launches": v[0], "avg_us": 1e3 * v[1] / v[0]} for k, v in sorted(prof.items())}
    by_kernel = {}
    for k, rec in kernels.items():
        kind = kernel_kind(k)
        if kind and kind in model:
            by_kernel[k] = dict(avg_us=rec["avg_us"], **bounds_of(model[kind], rec["avg_us"] * 1e-6, peaks, clock))
    if spans:
        for k, span in spans.items():
            if k in kernels and span > 0:
                kernels[k]["device_span_us"] = span
                if k in by_kernel:
                    by_kernel[k]["device_span_us"] = span
                    by_kernel[k]["frac_device_span"] = by_kernel[k]["frac"] * by_kernel[k]["avg_us"] / span
    dom = headline_kernel if headline_kernel in by_kernel else None
    if dom is None and by_kernel:
        dom = max((k for k in by_kernel if kernel_kind(k) in ("pass1", "pass2")), key=lambda k: kernels[k]["avg_us"], default=None)
    roof = {"kernel": dom, "launches": kernels[dom]["launches"] if dom else None, "traffic": None}
    if dom:
        roof.update(by_kernel[dom])
        roof["traffic"] = ncu_traffic(name, dom)
    roof["kernels"] = by_kernel
    roof["step"] = dict(us=ms_step * 1e3, **bounds_of(model["step"], ms_step * 1e-3, peaks, clock))
    line = {"metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "config": workload_config(name, world),
            "timing": {"rounds": rounds, "steps_per_round": args.steps, "reported": "median round",
                       "min_timed_s": MIN_TIMED_S, "launch": launch,
                       # the first rounds run at boost clocks; under a long run the power cap lowers them (see `clocks`)
                       "ms_per_step_of_rounds": {k: v / args.steps for k, v in (timing_detail or {}).items()}},
            "clocks": clocks, "e2e": e2e,
            "gpu_launches": (sum(v[0] for v in prof.values()) // max(prof_steps, 1)) * args.steps,
            "roofline": roof, "kernels": kernels, "cpu_baseline": cpu}
    if extra:
        line.update(extra)
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------
# CPU checker legs (bounded samples of each workload)
# ---------------------------------------------------------------------------------------------------
def cpu_prefill_sample(case, run, *, heads=None, batch=None, given=False, adaptive=False, budget_s=10.0, max_reps=8):
    """The checker on a sample of `case`: KV heads [0, heads) of batch items [0, batch); score, pool + select,
    compact.  Returns (layer-equivalent tokens per second, description, seconds)."""
    import numpy as np
    from oracle import reference as ref
    ref.build()
    B = case.B if batch is None else batch
    H = case.Hkv if heads is None else heads
    G = case.G
    q, k, v = case.q[:B, :H * G], case.k[:B, :H], case.v[:B, :H]
    lens = case.seq_lens[:B]
    want = tuple(run["variants"])
    budgets = run["budget"] if isinstance(run["budget"], list) else [run["budget"]] * case.B
    stride = int(max(budgets)) * (4 if adaptive else 1)
    giv = None
    if given:                                  # the window attention a caller would hand over (untimed)
        out = ref.score(q, k, v, seq_lens=lens, want=("ATTN",), return_attention=True)
        giv = (out["O"].reshape(B, H * G, case.W, case.d).astype(np.float32),
               (out["m"] + np.log(out["l"])).reshape(B, H * G, case.W).astype(np.float32))
    reps, t0 = 0, time.time()
    while reps < 1 or (time.time() - t0 < budget_s and reps < max_reps):
        s = ref.score(q, k, v, seq_lens=lens, want=want, given=giv)[want[-1]].astype(np.float32)
        if adaptive:
            ridx, _ = ref.select_adaptive_pipeline(s, lens, budgets[:B], run["n_sink"], run["n_recent"], run["pool_mode"],
                                                   run["pool_kernel"], 0.2, stride)
        else:
            ridx = ref.select_pipeline(s, lens, budgets[:B], run["n_sink"], run["n_recent"], run["pool_mode"],
                                       run["pool_kernel"], stride)
        for b in range(B):
            for h in range(H):
                n, cnt = int(lens[b]), int((ridx[b, h] >= 0).sum())     # rows are padded with -1 beyond the kept tokens
                ref.compact(case.k_bits[b, h, :n], ridx[b, h, :cnt], cnt)
                ref.compact(case.v_bits[b, h, :n], ridx[b, h, :cnt], cnt)
        reps += 1
    dt = time.time() - t0
    tokens = int(lens.sum()) * (H / case.Hkv)            # layer-equivalent tokens (all KV heads of a layer)
    desc = (f"KV heads 0..{H - 1} of {case.Hkv}, batch items 0..{B - 1} of {case.B} ({int(lens.sum())} tokens per head), "
            f"{reps} repetition(s), {dt:.1f} s; scaled to one layer by the head count")
    return tokens * reps / dt, desc, dt


def cpu_decode_sample(dc, *, n0, budget, n_sink, n_recent, steps=8, window=0):
    """`steps` decode steps of the checker over every (batch item, KV head): append, W = 1 scores, accumulate, evict."""
    import numpy as np
    from oracle import reference as ref
    ref.build()
    B, Hkv, G, cap = dc.k0.shape[0], dc.k0.shape[1], dc.q_t.shape[2] // dc.k0.shape[1], budget + 1
    sts = [[ref.DecodeState(dc.k0[b, h], dc.v0[b, h], cap, window=window) for h in range(Hkv)] for b in range(B)]
    t0 = time.time()
    for t in range(steps):
        for b in range(B):
            for h in range(Hkv):
                st = sts[b][h]
                st.append(dc.k_t[t, b, h], dc.v_t[t, b, h], n0 + t)
                acc = st.accumulate(st.scores(dc.q_t[t, b, h * G:(h + 1) * G], "VK"), n0 + t)
                live = st.pos >= 0
                st.s_acc[live] = acc[live].astype(np.float32)
                st.evict(n0 + t, budget, n_sink, n_recent)
    dt = time.time() - t0
    return steps / dt, f"{steps} steps over all {B} x {Hkv} heads ({n0 + 1} live slots each), {dt:.1f} s", dt


# ---------------------------------------------------------------------------------------------------
# reference arm: the CPU checker
# ---------------------------------------------------------------------------------------------------
def run_reference(args):
    """The CPU checker as it stands, timed on the host cores (rank 0 only).  Each step is a bounded sample of
    the workload, sized so that the whole run ends within a few minutes; the value is scaled to the metric's unit."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import reference as ref
    from paper_2510_07651_b200 import synth
    ref.build()
    cores = ref.host_threads()
    name = args.workload
    per_step = 120.0 / (args.steps + args.warmup)
    if name.startswith("decode"):
        n0, budget = 4096, 4096
        dc = synth.make_decode(B=32, Hq=32, Hkv=8, d=128, n0=n0, steps=args.steps + args.warmup, seed=1239)
        window = 16 if name == "decode-window" else 0
        val, desc, dt = cpu_decode_sample(dc, n0=n0, budget=budget, n_sink=4, n_recent=256,
                                          steps=min(max(1, args.steps), dc.q_t.shape[0]), window=window)
        value, metric, unit, ms_step, sample = val, "decode rescoring steps/sec", "steps/s", 1e3 / val, desc
    else:
        base = name.replace("-given", "").replace("-adaptive", "").replace("-sharded", "")
        case, run = synth.full_history(4096) if base == "history4k" else synth.config(PREFILL[base], seed=1236 if base == "llama32k" else None)
        given, adaptive = name.endswith("-given"), name.endswith("-adaptive")
        # size the sample: time one KV head of one batch item, then take as many heads (and batch items) as fit a step
        heads, batch = 1, 1
        v0, _, dt0 = cpu_prefill_sample(case, run, heads=1, batch=1, given=given, adaptive=adaptive, budget_s=0.0, max_reps=1)
        per_head_s = dt0
        heads = int(max(1, min(case.Hkv, per_step / max(per_head_s, 1e-3))))
        if heads == case.Hkv and case.B > 1:
            batch = int(max(1, min(case.B, per_step / max(per_head_s * case.Hkv, 1e-3))))
        for _ in range(args.warmup):
            cpu_prefill_sample(case, run, heads=heads, batch=batch, given=given, adaptive=adaptive, budget_s=0.0, max_reps=1)
        t0, tok = time.time(), 0.0
        for _ in range(args.steps):
            v, sample, dt = cpu_prefill_sample(case, run, heads=heads, batch=batch, given=given, adaptive=adaptive, budget_s=0.0, max_reps=1)
            tok += v * dt
        total = time.time() - t0
        value, metric, unit, ms_step = tok / total, METRIC, UNIT, 1e3 * total / args.steps
        sample = sample.split(", 1 repetition")[0] + " per step; scaled to one layer by the head count"
    line = {"impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(name, args.gpus),
            "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------
# the library arm
# ---------------------------------------------------------------------------------------------------
def setup_gpu():
    import torch
    import torch.distributed as dist
    from paper_2510_07651_b200 import api, build
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    api.lib()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
    return world, rank, local, barrier


def run_prefill(args):
    """llama32k (the headline), qwen128k, ragged, their -given / -adaptive variants and history4k."""
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2510_07651_b200 import api, synth

    name = args.workload
    world, rank, local, barrier = setup_gpu()
    if world > 1 and name != "llama32k":
        raise SystemExit("only the headline workload runs on several GPUs")
    peaks = load_peaks()
    given, adaptive = name.endswith("-given"), name.endswith("-adaptive")
    base = name.replace("-given", "").replace("-adaptive", "")
    headline = name == "llama32k"
    n_copies = {"llama32k": 4, "history4k": 16}.get(base, 1)

    bf = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    cases, dev = [], []
    for c in range(n_copies):
        if base == "history4k":
            case, run = synth.full_history(4096, seed=1240 + c)
        elif base == "llama32k":
            case, run = synth.config(2, seed=1236 + 100 * rank + c)
        else:
            case, run = synth.config(PREFILL[base])
        cases.append(case)
        dev.append((bf(case.q_bits), bf(case.k_bits), bf(case.v_bits)))
    case = cases[0]
    B, Hkv, N, d = case.B, case.Hkv, case.Nmax, case.d
    tokens_per_step = int(case.seq_lens.sum())
    lens = None if (case.seq_lens == case.Nmax).all() else torch.from_numpy(case.seq_lens).cuda()
    order = [n for n in ("V", "K", "VK") if n in run["variants"]]
    budgets = np.asarray(run["budget"] if isinstance(run["budget"], list) else [run["budget"]] * B, np.int32)
    uniform = bool((budgets == budgets[0]).all())
    bud_d = None if uniform else torch.from_numpy(budgets).cuda()
    stride = int(budgets.max()) * (4 if adaptive else 1)      # adaptive: a head may keep up to four average budgets

    # ---- preallocated outputs and workspaces (nothing is allocated inside the timed region) -----
    sp = api.score_params(dev[0][0], dev[0][1], seq_lens=lens, variants=order, path=args.path)
    ws_score = torch.empty(api.obc_score_workspace(sp), dtype=torch.uint8, device="cuda")
    scores = torch.empty((len(order), B, Hkv, N), dtype=torch.float32, device="cuda")
    selp = api.select_params(scores[-1], budget=int(budgets[0]) if uniform else 0, budgets=bud_d, idx_stride=stride,
                             seq_lens=lens, n_recent=run["n_recent"], pool=run["pool_mode"], pool_kernel=run["pool_kernel"])
    ws_sel = torch.empty(api.obc_select_workspace(selp), dtype=torch.uint8, device="cuda")
    if adaptive:
        n_ws = api.C.c_size_t(0)
        api._check(api.lib().obc_select_adaptive_workspace(api.C.byref(selp), 0.2, api.C.byref(n_ws)), "obc_select_adaptive_workspace")
        ws_sel = torch.empty(n_ws.value, dtype=torch.uint8, device="cuda")
    counts = torch.empty((B, Hkv), dtype=torch.int32, device="cuda")
    idx = torch.empty((B, Hkv, stride), dtype=torch.int32, device="cuda")
    k_out = torch.empty((B, Hkv, stride, d), dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)

    given_dev = []
    if given:
        # what the model's attention kernel would hand over for the window rows, made here (untimed set-up)
        # with plain tensor ops: O = softmax(scale * Q K^T) V and the natural-log LSE, causal over the window
        G, W, scale = case.G, case.W, 1.0 / np.sqrt(128.0)
        for (q, k, v) in dev:
            o_win = torch.empty((B, case.Hq, W, 128), dtype=torch.bfloat16, device="cuda")
            lse_win = torch.empty((B, case.Hq, W), dtype=torch.float32, device="cuda")
            for b_ in range(B):
                n = int(case.seq_lens[b_])
                vis = torch.arange(n, device="cuda")[None, :] <= (n - W + torch.arange(W, device="cuda"))[:, None]
                for g_ in range(Hkv):
                    qg = q[b_, g_ * G:(g_ + 1) * G].float()
                    z = torch.einsum("gwd,nd->gwn", qg, k[b_, g_, :n].float()) * scale
                    z = z.masked_fill(~vis[None], float("-inf"))
                    lse_win[b_, g_ * G:(g_ + 1) * G] = torch.logsumexp(z, dim=-1)
                    o_win[b_, g_ * G:(g_ + 1) * G] = (torch.softmax(z, dim=-1) @ v[b_, g_, :n].float()).to(torch.bfloat16)
                    del z
            given_dev.append((o_win, lse_win))
        torch.cuda.synchronize()

    def step_on(q, k, v, c, oi=idx, ok=k_out, ov=v_out):
        if given:
            api.obc_score_given(q, k, v, given_dev[c][0], given_dev[c][1], seq_lens=lens, variants=order, scores=scores,
                                workspace=ws_score)
        else:
            api.obc_score(q, k, v, seq_lens=lens, variants=order, path=args.path, scores=scores, workspace=ws_score)
        if adaptive:
            api.obc_select_adaptive(scores[-1], budget=int(budgets[0]), safeguard=0.2, idx_stride=stride, seq_lens=lens,
                                    n_recent=run["n_recent"], pool=run["pool_mode"], pool_kernel=run["pool_kernel"],
                                    idx=oi, counts=counts, workspace=ws_sel)
        else:
            api.obc_select(scores[-1], budget=int(budgets[0]) if uniform else 0, budgets=bud_d, idx_stride=stride,
                           seq_lens=lens, n_recent=run["n_recent"], pool=run["pool_mode"], pool_kernel=run["pool_kernel"],
                           idx=oi, workspace=ws_sel)
        api.obc_compact(k, v, oi, k_out=ok, v_out=ov)

    def step(i):
        c = i % n_copies
        step_on(*dev[c], c)

    # One CUDA graph per input copy holds the whole step (the library only enqueues work on the
    # current stream and allocates nothing, so a step can be captured); both ways of issuing a step
    # are timed, plain library calls and graph replay; the job's figure is the faster one.
    for i in range(n_copies):
        step(i)                                     # first calls: function attributes, lazy module load
    torch.cuda.synchronize()
    graphs = []
    if not args.eager:
        for i in range(n_copies):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                step(i)
            graphs.append(g)

    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.mark("timed_begin")
    by_mode = {"plain library calls": time_rounds(step, args.steps, args.warmup, barrier)}
    detail = {"plain library calls": dict(time_rounds.last)}
    if graphs:
        by_mode["one captured CUDA graph per step, replayed"] = time_rounds(lambda i: graphs[i % n_copies].replay(),
                                                                            args.steps, args.warmup, barrier)
        detail["one captured CUDA graph per step, replayed"] = dict(time_rounds.last)
    if sampler:
        sampler.mark("timed_end")
    launch_mode, (ms_round, rounds) = min(by_mode.items(), key=lambda kv: kv[1][0])

    # ---- per-kernel times (same steps again, every kernel bracketed by CUDA events) -------------
    prof_steps = max(20, min(args.steps, 200))
    api.obc_profile_begin()
    for i in range(prof_steps):
        step(i)
    torch.cuda.synchronize()
    prof = api.obc_profile_end()
    clocks = sampler.stop() if sampler else None

    # ---- device-side extents of the two tensor-core score kernels (first CTA start to last CTA end, read from
    # the GPU's own timer by the kernels): plain calls, one step at a time, no events between the kernels ----
    api.obc_score_kernel_spans(ws_score)                # zeroes the header words
    spans = {"tc_pass1": 0.0, "tc_pass2": 0.0}
    span_steps = 20
    for i in range(span_steps):
        step(i)
        s1, s2 = api.obc_score_kernel_spans(ws_score)
        spans["tc_pass1"] += s1 / span_steps; spans["tc_pass2"] += s2 / span_steps

    e2e = None
    if headline:
        e2e = run_e2e(args, world, barrier, dev, step_on, idx, k_out, v_out, tokens_per_step)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = None
    if world == 1 and not args.no_cpu:
        if base == "llama32k":
            v, desc, _ = cpu_prefill_sample(case, run, given=given, adaptive=adaptive)
        elif base == "ragged":
            v, desc, _ = cpu_prefill_sample(case, run, batch=1, budget_s=10.0, max_reps=2)
        else:                                   # qwen128k, history4k: one KV head
            v, desc, _ = cpu_prefill_sample(case, run, heads=1, given=given, budget_s=10.0, max_reps=2)
        from oracle import reference as ref
        cpu = {"value": v, "unit": UNIT, "cores": ref.host_threads(), "kind": "oracle", "sample": desc}

    value = world * tokens_per_step * args.steps / (ms_round * 1e-3)
    finish_line(name=name, world=world, args=args, metric=METRIC, unit=UNIT, value=value, ms_round=ms_round, rounds=rounds,
                prof=prof, prof_steps=prof_steps, model=prefill_model(case, run, given), peaks=peaks, clocks=clocks, cpu=cpu,
                e2e=e2e, headline_kernel="tc_pass2", spans=spans, launch=launch_mode, timing_detail=detail[launch_mode],
                extra={"ms_per_step_by_launch": {k: v[0] / args.steps for k, v in by_mode.items()}, "path": args.path})
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, world, barrier, dev, step_on, idx, k_out, v_out, tokens_per_step):
    """End to end: host (pinned) inputs -> device, the whole path, results back to the host, every step.
    The caller double-buffers, as a serving loop would: while step i runs, the inputs of step i + 1 travel to the
    device on a copy stream and the results of step i - 1 travel back on another."""
    import torch
    import torch.distributed as dist
    pin = lambda t: t.cpu().pin_memory()
    host = [tuple(pin(t) for t in dev[c]) for c in range(2)]
    h2d = sum(t.numel() * t.element_size() for t in host[0])
    d2h = sum(t.numel() * t.element_size() for t in (idx, k_out, v_out))
    dins = [tuple(torch.empty_like(t) for t in dev[0]) for _ in range(2)]
    houts = [(pin(idx), pin(k_out), pin(v_out)) for _ in range(2)]
    douts = [(idx, k_out, v_out), tuple(torch.empty_like(t) for t in (idx, k_out, v_out))]
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]           # inputs of buffer b have arrived
    ev_free = [torch.cuda.Event() for _ in range(2)]         # the step that read input buffer b has run
    ev_done = [torch.cuda.Event() for _ in range(2)]         # results of buffer b are complete on the device
    ev_back = [torch.cuda.Event() for _ in range(2)]         # results of buffer b are on the host

    def e2e_run(n):
        for b in range(2):
            ev_free[b].record(main); ev_back[b].record(s_out)
        for i in range(n + 1):
            b = i % 2
            if i < n:                                        # inputs of step i: host -> device
                s_in.wait_event(ev_free[b])
                with torch.cuda.stream(s_in):
                    for d_, h_ in zip(dins[b], host[b]):
                        d_.copy_(h_, non_blocking=True)
                    ev_in[b].record(s_in)
            if i > 0:                                        # step i - 1 on the main stream, its results device -> host
                pb = (i - 1) % 2
                main.wait_event(ev_in[pb]); main.wait_event(ev_back[pb])
                step_on(*dins[pb], pb, *douts[pb])
                ev_free[pb].record(main); ev_done[pb].record(main)
                s_out.wait_event(ev_done[pb])
                with torch.cuda.stream(s_out):
                    for h_, d_ in zip(houts[pb], douts[pb]):
                        h_.copy_(d_, non_blocking=True)
                    ev_back[pb].record(s_out)
            if i > 1:
                ev_back[i % 2].synchronize()                 # the caller reads the results of step i - 2
        ev_back[(n - 1) % 2].synchronize()

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = max(3, min(args.steps, 20))
    e2e_run(2)
    barrier()
    t0 = time.perf_counter()
    e0.record()
    e2e_run(e2e_steps)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = torch.tensor([max(e0.elapsed_time(e1), 1e3 * (time.perf_counter() - t0))], device="cuda")
    last = (e2e_steps - 1) % 2                              # what came back is what a plain step gives for those inputs
    got_idx, got_k = houts[last][0].clone(), houts[last][1].clone()
    step_on(*dev[last], last)
    torch.cuda.synchronize()
    if not (torch.equal(got_idx, idx.cpu()) and torch.equal(got_k.view(torch.int16), k_out.cpu().view(torch.int16))):
        raise RuntimeError("end-to-end run: the results copied back differ from a plain step on the same inputs")
    if world > 1:
        dist.all_reduce(e2e_ms, op=dist.ReduceOp.MAX)
    return {"value": world * tokens_per_step * e2e_steps / (float(e2e_ms.item()) * 1e-3), "unit": UNIT,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}


def run_decode(args):
    """Llama-3-8B shapes, batch 32: a 16384-token context already reduced to the 4096-token budget;
    every step appends one token, rescores all 4097 live slots (W = 1) and evicts one."""
    import numpy as np
    import torch
    from paper_2510_07651_b200 import api, synth
    world, rank, local, barrier = setup_gpu()
    peaks = load_peaks()
    bf = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    B, Hq, Hkv, n0, budget, n_sink, n_recent = 32, 32, 8, 4096, 4096, 4, 256
    dc = synth.make_decode(B=B, Hq=Hq, Hkv=Hkv, d=128, n0=n0, steps=64, seed=1239)
    cap = budget + 1
    kc = torch.zeros((B, Hkv, cap, 128), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    kc[:, :, :n0] = bf(dc.k0_bits); vc[:, :, :n0] = bf(dc.v0_bits)
    pos = torch.full((B, Hkv, cap), -1, dtype=torch.int32, device="cuda")
    pos[:, :, :n0] = torch.arange(n0, dtype=torch.int32, device="cuda")
    s_acc = torch.zeros((B, Hkv, cap), dtype=torch.float32, device="cuda")
    state = torch.zeros((B, Hkv, 4), dtype=torch.int32, device="cuda")
    state[..., 0] = n0; state[..., 1] = n0; state[..., 2] = n0
    qd, kd, vd = bf(dc.q_t_bits), bf(dc.k_t_bits), bf(dc.v_t_bits)
    ns = qd.shape[0]
    q_t = [qd[t].unsqueeze(2) for t in range(ns)]; k_t = [kd[t].unsqueeze(2) for t in range(ns)]
    v_t = [vd[t].unsqueeze(2) for t in range(ns)]
    p = api.decode_params(q_t[0], kc, budget=budget, n_sink=n_sink, n_recent=n_recent)
    ws = torch.empty(api.obc_decode_workspace(p), dtype=torch.uint8, device="cuda")
    window = 16 if args.workload == "decode-window" else 0       # scores accumulated over the last 16 steps only
    hist = torch.zeros((B, Hkv, window, cap), dtype=torch.float32, device="cuda") if window else None

    def step(t):
        api.obc_decode_step(q_t[t % ns], k_t[t % ns], v_t[t % ns], kc, vc, s_acc, pos, state, n0 + t,
                            budget=budget, n_sink=n_sink, n_recent=n_recent, variant="VK", workspace=ws,
                            acc_window=window, s_hist=hist)
    sampler = ClockSampler(local)
    sampler.mark("timed_begin")
    ms_round, rounds = time_rounds(step, args.steps, args.warmup, barrier)
    detail = dict(time_rounds.last)
    sampler.mark("timed_end")
    prof_steps = max(20, min(args.steps, 100))
    api.obc_profile_begin()
    for t in range(10 ** 6, 10 ** 6 + prof_steps):
        step(t)
    torch.cuda.synchronize()
    prof = api.obc_profile_end()
    clocks = sampler.stop()
    units, live = B * Hkv, n0 + 1
    pairs = units * live * (Hq // Hkv)
    kv = units * live * 128 * 2 * 2
    model = {"pass1": dict(bytes=kv, pairs=pairs, fp32_per_pair=5, ex2_per_pair=1),
             "step": dict(bytes=units * live * 520, flops=0, pairs=pairs, fp32_per_pair=15, ex2_per_pair=2)}
    cpu = None
    if not args.no_cpu:
        from oracle import reference as ref
        v, desc, _ = cpu_decode_sample(dc, n0=n0, budget=budget, n_sink=n_sink, n_recent=n_recent, steps=8, window=window)
        cpu = {"value": v, "unit": "steps/s", "cores": ref.host_threads(), "kind": "oracle", "sample": desc}
    finish_line(name=args.workload, world=1, args=args, metric="decode rescoring steps/sec", unit="steps/s",
                value=args.steps / (ms_round * 1e-3), ms_round=ms_round, rounds=rounds, prof=prof, prof_steps=prof_steps,
                model=model, peaks=peaks, clocks=clocks, cpu=cpu, launch="plain library calls", timing_detail=detail,
                extra={"note": "the step's algorithmic bytes are the floor (K and V of every live slot once, 8 bytes of "
                               "accumulator and position traffic per slot); the kernels read V twice"})


def run_sharded(args):
    """One rank's share of the 32k Llama layer sharded by token range over two ranks (context parallelism):
    this rank holds the second half of the tokens (the window's own tokens are among them).  Per step: the shard's
    window attention, the merge with the other rank's (o, lse) (computed once during set-up; in a real job it arrives
    by all-gather: B*Hq*W*(d+1) floats = 0.5 MB), the scores of the local tokens, and the selection over the whole
    sequence's scores (the other half filled in once during set-up)."""
    import numpy as np
    import torch
    from paper_2510_07651_b200 import api, synth
    world, rank, local, barrier = setup_gpu()
    peaks = load_peaks()
    bf = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    n_copies = 4
    sets = []
    for c in range(n_copies):
        case, run = synth.config(2, seed=1236 + c)
        q, k, v = bf(case.q_bits), bf(case.k_bits), bf(case.v_bits)
        N, half = case.Nmax, case.Nmax // 2
        m0 = torch.full((case.B,), N, dtype=torch.int32, device="cuda")
        m1 = torch.full((case.B,), N - half, dtype=torch.int32, device="cuda")
        k0, v0, k1, v1 = k[:, :, :half], v[:, :, :half], k[:, :, half:], v[:, :, half:]
        o_parts = torch.empty((2, case.B, case.Hq, case.W, 128), dtype=torch.float32, device="cuda")
        lse_parts = torch.empty((2, case.B, case.Hq, case.W), dtype=torch.float32, device="cuda")
        api.obc_window_attention(q, k0, v0, mask_lens=m0, o_out=o_parts[0], lse_out=lse_parts[0])
        sets.append(dict(q=q, k1=k1, v1=v1, m1=m1, o_parts=o_parts, lse_parts=lse_parts))
        if c == 0:
            o_all, lse_all = torch.empty_like(o_parts[0]), torch.empty_like(lse_parts[0])
            sp = api.score_params(q, k1, variants=["VK"], mask_lens=m1)
            ws = torch.empty(api.obc_score_workspace(sp), dtype=torch.uint8, device="cuda")
            scores = torch.zeros((1, case.B, case.Hkv, N), dtype=torch.float32, device="cuda")
            loc = torch.empty((1, case.B, case.Hkv, N - half), dtype=torch.float32, device="cuda")
            selp = api.select_params(scores[0], budget=run["budget"], n_recent=run["n_recent"], pool=run["pool_mode"],
                                     pool_kernel=run["pool_kernel"])
            ws_sel = torch.empty(api.obc_select_workspace(selp), dtype=torch.uint8, device="cuda")
            idx = torch.empty((case.B, case.Hkv, run["budget"]), dtype=torch.int32, device="cuda")
            api.obc_window_attention(q, k1, v1, mask_lens=m1, o_out=o_parts[1], lse_out=lse_parts[1], workspace=ws)
            api.obc_merge_attention(o_parts, lse_parts, o_out=o_all, lse_out=lse_all)
            sp0 = api.score_params(q, k0, variants=["VK"], mask_lens=m0)
            ws0 = torch.empty(api.obc_score_workspace(sp0), dtype=torch.uint8, device="cuda")
            scores[..., :half] = api.obc_score_given(q, k0, v0, o_all, lse_all, variants=["VK"], mask_lens=m0, workspace=ws0)
    torch.cuda.synchronize()

    def step(i):
        s = sets[i % n_copies]
        api.obc_window_attention(s["q"], s["k1"], s["v1"], mask_lens=s["m1"], o_out=s["o_parts"][1], lse_out=s["lse_parts"][1], workspace=ws)
        api.obc_merge_attention(s["o_parts"], s["lse_parts"], o_out=o_all, lse_out=lse_all)
        api.obc_score_given(s["q"], s["k1"], s["v1"], o_all, lse_all, variants=["VK"], mask_lens=s["m1"], scores=loc, workspace=ws)
        scores[..., half:].copy_(loc)                       # stands for the all-gather of the scores
        api.obc_select(scores[0], budget=run["budget"], n_recent=run["n_recent"], pool=run["pool_mode"],
                       pool_kernel=run["pool_kernel"], idx=idx, workspace=ws_sel)
    sampler = ClockSampler(local)
    sampler.mark("timed_begin")
    ms_round, rounds = time_rounds(step, args.steps, args.warmup, barrier)
    detail = dict(time_rounds.last)
    sampler.mark("timed_end")
    prof_steps = max(20, min(args.steps, 50))
    api.obc_profile_begin()
    for i in range(prof_steps):
        step(i)
    torch.cuda.synchronize()
    prof = api.obc_profile_end()
    clocks = sampler.stop()
    tok_heads = (N - half) * case.Hkv
    pairs = sum(N - half - case.W + i + 1 for i in range(case.W)) * case.G * case.Hkv
    kv = tok_heads * 512
    model = {"pass1": dict(bytes=kv, flops=4 * 128 * pairs, pairs=pairs, fp32_per_pair=5, ex2_per_pair=1),
             "pass2": dict(bytes=kv + tok_heads * 4, flops=4 * 128 * pairs, pairs=pairs, fp32_per_pair=7, ex2_per_pair=1),
             "step": dict(bytes=2 * kv + tok_heads * 12 + N * case.Hkv * 4, flops=8 * 128 * pairs, pairs=2 * pairs, fp32_per_pair=6, ex2_per_pair=1)}
    cpu = None
    if not args.no_cpu:
        from oracle import reference as ref
        v, desc, _ = cpu_prefill_sample(case, run)
        cpu = {"value": v, "unit": UNIT, "cores": ref.host_threads(), "kind": "oracle",
               "sample": "the unsharded layer: " + desc}
    finish_line(name=args.workload, world=1, args=args, metric=METRIC, unit=UNIT, value=N * args.steps / (ms_round * 1e-3),
                ms_round=ms_round, rounds=rounds, prof=prof, prof_steps=prof_steps, model=model, peaks=peaks, clocks=clocks,
                cpu=cpu, launch="plain library calls", timing_detail=detail,
                extra={"note": "the step's algorithmic bytes count the shard's K and V twice: with the attention merged across "
                               "ranks between the passes, the second read cannot be saved"})


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--path", default="auto", choices=["auto", "simt", "tc"])
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-baseline leg")
    ap.add_argument("--eager", action="store_true", help="time plain library calls only (no CUDA graph replay)")
    ap.add_argument("--min-timed-s", type=float, default=None,
                    help="timed rounds are repeated until this many seconds are timed (default 0.5; 0 = one round, for profiler runs)")
    ap.add_argument("--workload", default="llama32k", choices=WORKLOADS,
                    help="llama32k is the headline benchmark (the only one that runs on several GPUs)")
    args = ap.parse_args()
    ref_arm = args.impl == "reference"
    if args.min_timed_s is not None:
        global MIN_TIMED_S
        MIN_TIMED_S = max(0.0, args.min_timed_s)
    if args.steps is None:
        args.steps = 3 if ref_arm else (2000 if args.workload == "llama32k" else 200)
    if args.warmup is None:
        args.warmup = 1 if ref_arm else 20
    if not ref_arm:
        args.warmup = max(args.warmup, 3)
    if ref_arm:
        run_reference(args)
    elif args.workload.startswith("decode"):
        run_decode(args)
    elif args.workload == "llama32k-sharded":
        run_sharded(args)
    else:
        run_prefill(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the OBCache hot path (score -> pool/select -> compact) on B200.

A "step" is one pass of the whole path over one Llama-3-8B-shaped layer cache (32 query heads /
8 KV heads, head_dim 128, N = 32768 cached tokens, window W = 32, bf16, OBCache-V&K, max-pool 7,
budget 2048 per head).  The metric is cached tokens scored+compacted per second per layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 it is launched by torch.distributed.run, one rank per GPU; every rank processes its
own cache (the (batch, KV head) units are independent, so there is no data-path collective) and
the reported value is the sum over ranks divided by the slowest rank's time (weak scaling).

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
N_COPIES = 4            # distinct input copies rotated between steps (4 x 135 MB > 126 MB L2)


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
                                       "-lms", "50", "-i", str(device_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None
        self.marks = {}

    def mark(self, name):
        self.marks[name] = time.time()

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.06)
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
        where = "timed region"
        if not inside:                       # region shorter than the sampling period
            inside, where = parsed, "whole run"
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for x in inside for n, v in zip(names, x[4]) if v.strip() == "Active"})
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(x[1] for x in inside), "sm_max_mhz": inside[0][2],
                "power_w_max": max(x[3] for x in inside), "reasons": reasons, "samples": len(inside),
                "window": where}


def ncu_traffic(kernel):
    """DRAM bytes per launch of `kernel` from the committed ncu summary, or None when there is no
    capture or the kernel source has changed since it was taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "traffic.txt")
    if not os.path.exists(path):
        return None
    rec = dict(l.split() for l in open(path) if l.strip() and not l.startswith("#"))
    src = os.path.join(ROOT, "paper_2510_07651_b200", "csrc", "score_tc.cu")
    if rec.get("source_sha256") != hashlib.sha256(open(src, "rb").read()).hexdigest():
        return None
    return float(rec[kernel]) if kernel in rec else None


def make_case(seed):
    from paper_2510_07651_b200 import synth
    return synth.config(2, seed=seed)


def run_reference(args):
    """The CPU checker as it stands, timed on the host cores (rank 0 only).  Each step scores,
    selects and compacts a bounded sample of the workload: the first `heads` of the 8 KV heads
    (all 32768 tokens, all their query heads), sized so that the whole run ends within minutes."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np
    from oracle import reference as ref
    ref.build()
    case, run = make_case(1236)
    cores = ref.host_threads()
    G = case.G

    def step(heads, n_tok):
        q, k, v = case.q[:, :heads * G], case.k[:, :heads, :n_tok], case.v[:, :heads, :n_tok]
        s = ref.score(q, k, v, want=("VK",))["VK"].astype(np.float32)
        budget = min(run["budget"], n_tok)
        idx = ref.select_pipeline(s, np.array([n_tok], np.int32), [budget], 0, run["n_recent"], run["pool_mode"],
                                  run["pool_kernel"], budget)
        for h in range(heads):
            ref.compact(case.k_bits[0, h, :n_tok], idx[0, h], budget)
            ref.compact(case.v_bits[0, h, :n_tok], idx[0, h], budget)

    # size the per-step sample so that warm-up + timed steps take about two minutes in all
    t0 = time.time()
    step(1, 4096)
    t_unit = (time.time() - t0) / 4096                      # seconds per token of one KV head
    per_step = 120.0 / (args.steps + args.warmup)
    heads = int(max(1, min(case.Hkv, per_step / (t_unit * case.Nmax))))
    n_tok = case.Nmax
    if heads == 1 and t_unit * case.Nmax > per_step:
        n_tok = int(max(1024, min(case.Nmax, per_step / t_unit)) // 1024 * 1024)
    for _ in range(args.warmup):
        step(heads, n_tok)
    t0 = time.time()
    for _ in range(args.steps):
        step(heads, n_tok)
    dt = time.time() - t0
    value = n_tok * (heads / case.Hkv) * args.steps / dt           # layer-equivalent tokens per second
    sample = (f"{heads} of {case.Hkv} KV heads x the first {n_tok} of {case.Nmax} cached tokens per step, "
              "scaled to one layer (all 8 KV heads)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2510_07651_b200 import api, build, multirank, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    api.lib()
    peaks = load_peaks()

    # ---- inputs: N_COPIES distinct seeded caches, resident in HBM ------------------------------
    bf = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    cases, dev = [], []
    for c in range(N_COPIES):
        case, run = make_case(1236 + 100 * rank + c)
        cases.append(case)
        dev.append((bf(case.q_bits), bf(case.k_bits), bf(case.v_bits)))
    case = cases[0]
    B, Hkv, N, d, budget = case.B, case.Hkv, case.Nmax, case.d, run["budget"]
    tokens_per_step = int(case.seq_lens.sum())

    # ---- preallocated outputs and workspaces (nothing is allocated inside the timed region) -----
    sp = api.score_params(dev[0][0], dev[0][1], variants=run["variants"], path=args.path)
    ws_score = torch.empty(api.obc_score_workspace(sp), dtype=torch.uint8, device="cuda")
    scores = torch.empty((1, B, Hkv, N), dtype=torch.float32, device="cuda")
    selp = api.select_params(scores[0], budget=budget, n_recent=run["n_recent"], pool=run["pool_mode"],
                             pool_kernel=run["pool_kernel"])
    ws_sel = torch.empty(api.obc_select_workspace(selp), dtype=torch.uint8, device="cuda")
    idx = torch.empty((B, Hkv, budget), dtype=torch.int32, device="cuda")
    k_out = torch.empty((B, Hkv, budget, d), dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)

    def step(q, k, v):
        api.obc_score(q, k, v, variants=run["variants"], path=args.path, scores=scores, workspace=ws_score)
        api.obc_select(scores[0], budget=budget, n_recent=run["n_recent"], pool=run["pool_mode"],
                       pool_kernel=run["pool_kernel"], idx=idx, workspace=ws_sel)
        api.obc_compact(k, v, idx, k_out=k_out, v_out=v_out)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # One CUDA graph per input copy holds the whole step (the library only enqueues work on the
    # current stream and allocates nothing, so a step can be captured); the timed loop replays
    # them in rotation, which keeps the host out of the measurement.  --eager times plain calls.
    for i in range(N_COPIES):
        step(*dev[i])                               # first calls: function attributes, lazy module load
    torch.cuda.synchronize()
    graphs = []
    if not args.eager:
        for i in range(N_COPIES):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                step(*dev[i])
            graphs.append(g)

    # Both ways of issuing a step are timed over the same K steps, plain library calls and graph
    # replay; the job's figure is the faster one (which one wins depends on the host).
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(run):
        for i in range(args.warmup):
            run(i)
        barrier()
        e0.record()
        for i in range(args.steps):
            run(i)
        e1.record()
        torch.cuda.synchronize()
        barrier()
        return multirank.max_over_ranks(e0.elapsed_time(e1), "cuda")

    if sampler:
        sampler.mark("timed_begin")
    ms_by_mode = {"plain library calls": timed(lambda i: step(*dev[i % N_COPIES]))}
    if graphs:
        ms_by_mode["one captured CUDA graph per step, replayed"] = timed(lambda i: graphs[i % N_COPIES].replay())
    if sampler:
        sampler.mark("timed_end")
    launch_mode, ms = min(ms_by_mode.items(), key=lambda kv: kv[1])

    # ---- per-kernel times (same steps again, every kernel bracketed by CUDA events) -------------
    prof_steps = min(args.steps, 200)
    api.obc_profile_begin()
    for i in range(prof_steps):
        step(*dev[i % N_COPIES])
    torch.cuda.synchronize()
    prof = api.obc_profile_end()
    clocks = sampler.stop() if sampler else None
    launches_per_step = sum(v[0] for v in prof.values()) // max(prof_steps, 1)

    # ---- device-side extents of the two score kernels (first CTA start to last CTA end, read from the
    # GPU's own timer by the kernels): plain calls, one step at a time, no events between the kernels ----
    api.obc_score_kernel_spans(ws_score)                # zeroes the header words
    spans = [0.0, 0.0]
    span_steps = min(args.steps, 50)
    for i in range(span_steps):
        step(*dev[i % N_COPIES])
        s1, s2 = api.obc_score_kernel_spans(ws_score)
        spans[0] += s1 / span_steps; spans[1] += s2 / span_steps

    # ---- end to end: host (pinned) inputs -> device, whole path, results back to the host -------
    pin = lambda t: t.cpu().pin_memory()
    host = [tuple(pin(t) for t in dev[c]) for c in range(2)]
    dq, dk, dv = (torch.empty_like(t) for t in dev[0])
    h_idx, h_k, h_v = pin(idx), pin(k_out), pin(v_out)
    h2d = sum(t.numel() * t.element_size() for t in host[0])
    d2h = sum(t.numel() * t.element_size() for t in (h_idx, h_k, h_v))

    # The caller double-buffers, as a serving loop would: while step i runs, the inputs of step i + 1 travel to the
    # device on a copy stream and the results of step i - 1 travel back on another (PCIe carries both directions
    # at once).  Every step's inputs are copied in and every step's results are copied out and waited for.
    dins = [(dq, dk, dv), tuple(torch.empty_like(t) for t in dev[0])]
    houts = [(h_idx, h_k, h_v), (pin(idx), pin(k_out), pin(v_out))]
    douts = [(idx, k_out, v_out), tuple(torch.empty_like(t) for t in (idx, k_out, v_out))]
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]           # inputs of buffer b have arrived
    ev_free = [torch.cuda.Event() for _ in range(2)]         # the step that read input buffer b has run
    ev_done = [torch.cuda.Event() for _ in range(2)]         # results of buffer b are complete on the device
    ev_back = [torch.cuda.Event() for _ in range(2)]         # results of buffer b are on the host

    def e2e_step_buffers(b):
        oi, ok, ov = douts[b]
        api.obc_score(*dins[b], variants=run["variants"], path=args.path, scores=scores, workspace=ws_score)
        api.obc_select(scores[0], budget=budget, n_recent=run["n_recent"], pool=run["pool_mode"],
                       pool_kernel=run["pool_kernel"], idx=oi, workspace=ws_sel)
        api.obc_compact(dins[b][1], dins[b][2], oi, k_out=ok, v_out=ov)

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
                e2e_step_buffers(pb)
                ev_free[pb].record(main); ev_done[pb].record(main)
                s_out.wait_event(ev_done[pb])
                with torch.cuda.stream(s_out):
                    for h_, d_ in zip(houts[pb], douts[pb]):
                        h_.copy_(d_, non_blocking=True)
                    ev_back[pb].record(s_out)
            if i > 1:
                ev_back[i % 2].synchronize()                 # the caller reads the results of step i - 2
        ev_back[(n - 1) % 2].synchronize()

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
    step(*dev[last])
    torch.cuda.synchronize()
    if not (torch.equal(got_idx, idx.cpu()) and torch.equal(got_k.view(torch.int16), k_out.cpu().view(torch.int16))):
        raise RuntimeError("end-to-end run: the results copied back differ from a plain step on the same inputs")
    if world > 1:
        dist.all_reduce(e2e_ms, op=dist.ReduceOp.MAX)
    e2e_value = world * tokens_per_step * e2e_steps / (float(e2e_ms.item()) * 1e-3)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel -----------------------------------------------------------
    value = world * tokens_per_step * args.steps / (ms * 1e-3)
    dom = max(prof.items(), key=lambda kv: kv[1][1])
    dom_name, (dom_launches, dom_ms) = dom
    dom_avg_s = dom_ms * 1e-3 / dom_launches
    elem = 2
    R = case.R
    kv_bytes = B * Hkv * N * d * elem * 2                     # K and V read once
    alg = {   # algorithmic bytes / flops per launch of each kernel on this workload
        "pass1": (kv_bytes, 2 * 2 * R * N * d * B * Hkv),
        "pass2": (kv_bytes + B * Hkv * N * 4, 2 * 2 * R * N * d * B * Hkv),
    }
    kind = "pass2" if "pass2" in dom_name else "pass1" if "pass1" in dom_name else None
    roof = {"kernel": dom_name, "launches": dom_launches, "avg_us": dom_avg_s * 1e6, "traffic": None}
    if kind and dom_name.startswith("simt"):
        peak = 148 * 128 * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12      # fp32 FMA lanes x 2 flop x clock
        ach = alg[kind][1] / dom_avg_s / 1e12
        roof.update(bound="alu", achieved=ach, peak=peak, unit="TFLOP/s", frac=ach / peak,
                    peak_source="148 SMs x 128 fp32 lanes x 2 flop x max SM clock")
    elif kind:
        t_hbm = alg[kind][0] / (peaks["hbm_gbs"] * 1e9)
        t_mma = alg[kind][1] / (peaks["bf16_tflops_sustained"] * 1e12)
        if t_hbm >= t_mma:
            ach = alg[kind][0] / dom_avg_s / 1e9
            roof.update(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"],
                        peak_source=f"{peaks['source']} STREAM-style copy")
        else:
            ach = alg[kind][1] / dom_avg_s / 1e12
            roof.update(bound="tensor", achieved=ach, peak=peaks["bf16_tflops_sustained"], unit="TFLOP/s",
                        frac=ach / peaks["bf16_tflops_sustained"], peak_source=f"{peaks['source']} cuBLAS bf16 sustained")
    roof["traffic"] = ncu_traffic(dom_name)
    # the two streaming score kernels take nearly equal time; the same figures for both, whichever dominates
    by_kernel = {}
    for name, (n_l, ms_k) in prof.items():
        k2 = "pass2" if "pass2" in name else "pass1" if "pass1" in name else None
        if k2 and name.startswith("tc"):
            avg_s = ms_k * 1e-3 / n_l
            by_kernel[name] = {"avg_us": avg_s * 1e6, "algorithmic_bytes": alg[k2][0],
                               "achieved_gbs": alg[k2][0] / avg_s / 1e9, "frac": alg[k2][0] / avg_s / 1e9 / peaks["hbm_gbs"]}
    kernels = {k: {"launches": v[0], "avg_us": 1e3 * v[1] / v[0]} for k, v in sorted(prof.items())}
    # The event pair around a launch also times the launch latency that back-to-back kernels hide; the
    # kernels' own clock readings give the extent on the device, reported beside the event figure.
    for name, span in (("tc_pass1", spans[0]), ("tc_pass2", spans[1])):
        if name in kernels and span > 0:
            kernels[name]["device_span_us"] = span
            if name in by_kernel:
                by_kernel[name]["device_span_us"] = span
                by_kernel[name]["frac_device_span"] = by_kernel[name]["frac"] * by_kernel[name]["avg_us"] / span
            if name == dom_name and "achieved" in roof:
                roof["device_span_us"] = span
                roof["frac_device_span"] = roof["frac"] * roof["avg_us"] / span
    if by_kernel:
        roof["score_kernels"] = by_kernel

    # ---- CPU baseline: the checker as it stands, on this machine's host cores ----------------------
    cpu = None
    if world == 1 and not args.no_cpu:
        from oracle import reference as ref
        ref.build()
        c0 = cases[0]
        reps, t0 = 0, time.time()
        while reps < 1 or (time.time() - t0 < 10.0 and reps < 8):
            s = ref.score(c0.q, c0.k, c0.v, want=("VK",))["VK"].astype(np.float32)
            ridx = ref.select_pipeline(s, c0.seq_lens, [budget], 0, run["n_recent"], run["pool_mode"],
                                       run["pool_kernel"], budget)
            for h in range(Hkv):
                ref.compact(c0.k_bits[0, h], ridx[0, h], budget)
                ref.compact(c0.v_bits[0, h], ridx[0, h], budget)
            reps += 1
        dt = time.time() - t0
        cpu = {"value": tokens_per_step * reps / dt, "unit": UNIT, "cores": ref.host_threads(), "kind": "oracle",
               "sample": f"the full workload (8 KV heads x 32768 tokens), {reps} repetitions, {dt:.1f} s"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "path": args.path,
                       "launch": launch_mode,
                       "ms_per_step_by_launch": {k: v / args.steps for k, v in ms_by_mode.items()},
                       "l2": f"{N_COPIES} distinct input copies rotated between steps ({N_COPIES} x 135 MB > 126 MB L2)",
                       "parallelism": f"{world} independent layer caches, one per GPU, no collective"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roof, "kernels": kernels, "cpu_baseline": cpu}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_other(args):
    """The other workloads (parity-test cases, not the headline): one JSON line each with the step
    time from CUDA events and the per-kernel event times.  Single GPU."""
    import numpy as np
    import torch
    from paper_2510_07651_b200 import api, build, synth

    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    build.build()
    api.lib()
    bf = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    steps, warmup = args.steps, max(args.warmup, 3)

    if args.workload in ("decode", "decode-window"):
        # Llama-3-8B shapes, batch 32: a 16384-token context already reduced to the 4096-token budget;
        # every step appends one token, rescores all 4097 live slots (W = 1) and evicts one.
        B, Hq, Hkv, n0, budget, n_sink, n_recent = 32, 32, 8, 4096, 4096, 4, 256
        total = warmup + steps
        dc = synth.make_decode(B=B, Hq=Hq, Hkv=Hkv, d=128, n0=n0, steps=min(total, 64), seed=1239)
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
        for t in range(warmup):
            step(t)
        torch.cuda.synchronize()
        e0.record()
        for t in range(warmup, total):
            step(t)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        api.obc_profile_begin()
        for t in range(total, total + min(steps, 100)):
            step(t)
        torch.cuda.synchronize()
        prof = api.obc_profile_end()
        live_bytes = B * Hkv * (n0 + 1) * 128 * 2 * 3            # K once, V twice per step
        line = {"metric": "decode rescoring steps/sec", "value": steps / (ms * 1e-3), "unit": "steps/s",
                "ms_per_step": ms / steps, "steps": steps, "warmup": warmup, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": "decode: B32 Hq32 Hkv8 d128, live 4096 -> 4097 -> 4096 per step, W1, OBCache-V&K, "
                                       "4 sinks, 256 recent, one eviction per head per step"
                                       + (f", accumulator = the last {window} steps' scores" if window else "")},
                "hbm_gbs_algorithmic": live_bytes / (ms / steps * 1e-3) / 1e9,
                "kernels": {k: {"launches": v[0], "avg_us": 1e3 * v[1] / v[0]} for k, v in sorted(prof.items())}}
        print(json.dumps(line))
        return

    if args.workload == "llama32k-sharded":
        # One rank's share of the 32k Llama layer sharded by token range over two ranks (context parallelism):
        # this rank holds the second half of the tokens (the window's own tokens are among them).  Per step:
        # the shard's window attention, the merge with the other rank's (o, lse) (computed once during set-up;
        # in a real job it arrives by all-gather: B*Hq*W*(d+1) floats = 0.5 MB), the scores of the local tokens,
        # and the selection over the whole sequence's scores (the other half filled in once during set-up).
        case, run = synth.config(2)
        q, k, v = bf(case.q_bits), bf(case.k_bits), bf(case.v_bits)
        N, half = case.Nmax, case.Nmax // 2
        m0 = torch.full((case.B,), N, dtype=torch.int32, device="cuda")
        m1 = torch.full((case.B,), N - half, dtype=torch.int32, device="cuda")
        k0, v0, k1, v1 = k[:, :, :half], v[:, :, :half], k[:, :, half:], v[:, :, half:]
        o_parts = torch.empty((2, case.B, case.Hq, case.W, 128), dtype=torch.float32, device="cuda")
        lse_parts = torch.empty((2, case.B, case.Hq, case.W), dtype=torch.float32, device="cuda")
        api.obc_window_attention(q, k0, v0, mask_lens=m0, o_out=o_parts[0], lse_out=lse_parts[0])
        o_all, lse_all = torch.empty_like(o_parts[0]), torch.empty_like(lse_parts[0])
        sp = api.score_params(q, k1, variants=["VK"], mask_lens=m1)
        ws = torch.empty(api.obc_score_workspace(sp), dtype=torch.uint8, device="cuda")
        scores = torch.zeros((1, case.B, case.Hkv, N), dtype=torch.float32, device="cuda")
        loc = torch.empty((1, case.B, case.Hkv, N - half), dtype=torch.float32, device="cuda")
        api.obc_window_attention(q, k1, v1, mask_lens=m1, o_out=o_parts[1], lse_out=lse_parts[1], workspace=ws)
        api.obc_merge_attention(o_parts, lse_parts, o_out=o_all, lse_out=lse_all)
        sp0 = api.score_params(q, k0, variants=["VK"], mask_lens=m0)
        ws0 = torch.empty(api.obc_score_workspace(sp0), dtype=torch.uint8, device="cuda")
        scores[..., :half] = api.obc_score_given(q, k0, v0, o_all, lse_all, variants=["VK"], mask_lens=m0, workspace=ws0)
        selp = api.select_params(scores[0], budget=run["budget"], n_recent=run["n_recent"], pool=run["pool_mode"],
                                 pool_kernel=run["pool_kernel"])
        ws_sel = torch.empty(api.obc_select_workspace(selp), dtype=torch.uint8, device="cuda")
        idx = torch.empty((case.B, case.Hkv, run["budget"]), dtype=torch.int32, device="cuda")

        def step():
            api.obc_window_attention(q, k1, v1, mask_lens=m1, o_out=o_parts[1], lse_out=lse_parts[1], workspace=ws)
            api.obc_merge_attention(o_parts, lse_parts, o_out=o_all, lse_out=lse_all)
            api.obc_score_given(q, k1, v1, o_all, lse_all, variants=["VK"], mask_lens=m1, scores=loc, workspace=ws)
            scores[..., half:].copy_(loc)                       # stands for the all-gather of the scores
            api.obc_select(scores[0], budget=run["budget"], n_recent=run["n_recent"], pool=run["pool_mode"],
                           pool_kernel=run["pool_kernel"], idx=idx, workspace=ws_sel)
        for _ in range(warmup):
            step()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        api.obc_profile_begin()
        for _ in range(min(steps, 50)):
            step()
        torch.cuda.synchronize()
        prof = api.obc_profile_end()
        line = {"metric": METRIC, "value": N * steps / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms / steps,
                "steps": steps, "warmup": warmup, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": "one of two ranks of the 32k Llama layer sharded by token range (this rank: tokens "
                                       f"{half}..{N - 1}), emulated on one GPU: window attention of the shard, merge with the "
                                       "peer's (o, lse), local scores, selection over the gathered scores; no compaction",
                           "l2": "single input copy (K+V of the shard = 67 MB)"},
                "kernels": {k_: {"launches": v_[0], "avg_us": 1e3 * v_[1] / v_[0]} for k_, v_ in sorted(prof.items())}}
        print(json.dumps(line))
        return

    given = args.workload.endswith("-given")     # the caller's attention outputs instead of a recompute
    adaptive = args.workload.endswith("-adaptive")    # head-adaptive budgets (safeguard 0.2) instead of one budget per head
    if args.workload == "history4k":             # the whole sequence as perturbation window (W = N = 4096)
        case, run = synth.full_history(4096)
    else:
        idx_cfg = {"llama32k": 2, "qwen128k": 3, "ragged": 4}[args.workload.replace("-given", "").replace("-adaptive", "")]
        case, run = synth.config(idx_cfg)
    q, k, v = bf(case.q_bits), bf(case.k_bits), bf(case.v_bits)
    lens = None if (case.seq_lens == case.Nmax).all() else torch.from_numpy(case.seq_lens).cuda()
    order = [n for n in ("V", "K", "VK") if n in run["variants"]]
    budgets = np.asarray(run["budget"] if isinstance(run["budget"], list) else [run["budget"]] * case.B, np.int32)
    uniform = bool((budgets == budgets[0]).all())
    bud_d = None if uniform else torch.from_numpy(budgets).cuda()
    stride = int(budgets.max()) * (4 if adaptive else 1)      # adaptive: a head may keep up to four average budgets
    sp = api.score_params(q, k, seq_lens=lens, variants=order)
    ws_score = torch.empty(api.obc_score_workspace(sp), dtype=torch.uint8, device="cuda")
    scores = torch.empty((len(order), case.B, case.Hkv, case.Nmax), dtype=torch.float32, device="cuda")
    selp = api.select_params(scores[-1], budget=int(budgets[0]) if uniform else 0, budgets=bud_d, idx_stride=stride,
                             seq_lens=lens, n_recent=run["n_recent"], pool=run["pool_mode"], pool_kernel=run["pool_kernel"])
    ws_sel = torch.empty(api.obc_select_workspace(selp), dtype=torch.uint8, device="cuda")
    if adaptive:
        n_ws = api.C.c_size_t(0)
        api._check(api.lib().obc_select_adaptive_workspace(api.C.byref(selp), 0.2, api.C.byref(n_ws)), "obc_select_adaptive_workspace")
        ws_sel = torch.empty(n_ws.value, dtype=torch.uint8, device="cuda")
    counts = torch.empty((case.B, case.Hkv), dtype=torch.int32, device="cuda")
    idx = torch.empty((case.B, case.Hkv, stride), dtype=torch.int32, device="cuda")
    k_out = torch.empty((case.B, case.Hkv, stride, 128), dtype=torch.bfloat16, device="cuda")
    v_out = torch.empty_like(k_out)

    o_win = lse_win = None
    if given:
        # what the model's attention kernel would hand over for the window rows, made here (untimed set-up)
        # with plain tensor ops: O = softmax(scale * Q K^T) V and the natural-log LSE, causal over the window
        G, W, scale = case.G, case.W, 1.0 / np.sqrt(128.0)
        o_win = torch.empty((case.B, case.Hq, W, 128), dtype=torch.bfloat16, device="cuda")
        lse_win = torch.empty((case.B, case.Hq, W), dtype=torch.float32, device="cuda")
        for b_ in range(case.B):
            n = int(case.seq_lens[b_])
            vis = torch.arange(n, device="cuda")[None, :] <= (n - W + torch.arange(W, device="cuda"))[:, None]
            for g_ in range(case.Hkv):
                qg = q[b_, g_ * G:(g_ + 1) * G].float()                          # [G, W, d]
                z = torch.einsum("gwd,nd->gwn", qg, k[b_, g_, :n].float()) * scale
                z = z.masked_fill(~vis[None], float("-inf"))
                lse_win[b_, g_ * G:(g_ + 1) * G] = torch.logsumexp(z, dim=-1)
                o_win[b_, g_ * G:(g_ + 1) * G] = (torch.softmax(z, dim=-1) @ v[b_, g_, :n].float()).to(torch.bfloat16)
                del z
        torch.cuda.synchronize()

    def step():
        if given:
            api.obc_score_given(q, k, v, o_win, lse_win, seq_lens=lens, variants=order, scores=scores, workspace=ws_score)
        else:
            api.obc_score(q, k, v, seq_lens=lens, variants=order, scores=scores, workspace=ws_score)
        if adaptive:
            api.obc_select_adaptive(scores[-1], budget=int(budgets[0]), safeguard=0.2, idx_stride=stride, seq_lens=lens,
                                    n_recent=run["n_recent"], pool=run["pool_mode"], pool_kernel=run["pool_kernel"],
                                    idx=idx, counts=counts, workspace=ws_sel)
        else:
            api.obc_select(scores[-1], budget=int(budgets[0]) if uniform else 0, budgets=bud_d, idx_stride=stride,
                           seq_lens=lens, n_recent=run["n_recent"], pool=run["pool_mode"], pool_kernel=run["pool_kernel"],
                           idx=idx, workspace=ws_sel)
        api.obc_compact(k, v, idx, k_out=k_out, v_out=v_out)
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()               # the library allocates nothing and only enqueues: a step can be captured
    with torch.cuda.graph(graph):
        step()

    def timed(run):
        for _ in range(warmup):
            run()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            run()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)
    ms_by_mode = {"plain library calls": timed(step), "one captured CUDA graph per step, replayed": timed(graph.replay)}
    launch_mode, ms = min(ms_by_mode.items(), key=lambda kv: kv[1])
    api.obc_profile_begin()
    for _ in range(min(steps, 50)):
        step()
    torch.cuda.synchronize()
    prof = api.obc_profile_end()
    tokens = int(case.seq_lens.sum())
    line = {"metric": METRIC, "value": tokens * steps / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms / steps,
            "steps": steps, "warmup": warmup, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{case.name}: B{case.B} Hq{case.Hq} Hkv{case.Hkv} d128 Nmax{case.Nmax} W{case.W} bf16, "
                                   f"variants {order}, pool {run['pool_mode']} {run['pool_kernel']}, tokens/step {tokens}"
                                   + (", window O and LSE supplied by the caller (no recompute)" if given else "")
                                   + (", head-adaptive budgets (safeguard 0.2)" if adaptive else ""),
                       "launch": launch_mode, "ms_per_step_by_launch": {k_: v_ / steps for k_, v_ in ms_by_mode.items()},
                       "l2": "inputs (K+V) larger than L2" if tokens * case.Hkv * 512 > 126e6 else "single input copy"},
            "kernels": {k: {"launches": v[0], "avg_us": 1e3 * v[1] / v[0]} for k, v in sorted(prof.items())}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--path", default="auto", choices=["auto", "simt", "tc"])
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-baseline leg")
    ap.add_argument("--eager", action="store_true", help="time plain library calls instead of replaying CUDA graphs")
    ap.add_argument("--workload", default="llama32k", choices=["llama32k", "qwen128k", "ragged", "decode", "llama32k-given", "qwen128k-given", "llama32k-adaptive", "history4k", "decode-window", "llama32k-sharded"],
                    help="llama32k is the headline benchmark; the others print a shorter line (1 GPU)")
    args = ap.parse_args()
    ref_arm = args.impl == "reference"
    if args.steps is None:
        args.steps = 3 if ref_arm else (2000 if args.workload == "llama32k" else 200)
    if args.warmup is None:
        args.warmup = 1 if ref_arm else 20
    if not ref_arm:
        args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    elif args.workload != "llama32k":
        run_other(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

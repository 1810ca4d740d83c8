#!/usr/bin/env python
"""Benchmark of the Fathom decode-step hot path on B200.

One "step" is one decode step of one synthetic Qwen3-8B-shaped layer:
    fathom_alloc_depth -> fathom_scan -> fathom_topk -> fathom_sparse_attend
at n = 1,048,576 tokens, 8 KV heads / 32 query heads, d = 128, budget B = 48, k = 4096, planes in HBM
(the million-token configuration the metric is quoted on).  fathom_build_planes runs once per sequence,
before the steps, and is timed on its own (once_per_sequence).  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

--impl reference times the CPU oracle (oracle/, numpy fp64, as it stands) on a bounded sample of the
same workload on the host cores; it is a deliberately slow baseline, not a target.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2609_17652_b200 import dist as fdist

METRIC = "keys_scanned_per_s"
UNIT = "keys/s"
N_LAYERS = 4                                                    # layer stores a session's steps rotate over
WORKLOAD = dict(name="million-token session, one Qwen3-8B-shaped layer (config 3, planes in HBM)",
                n=1 << 20, Hkv=8, Hq=32, d=128, B=48, k=4096, heads_per_plan=4)
# dram__bytes_read.sum + dram__bytes_write.sum per unit (one token of one KV head) from the ncu captures
# summarised under profiles/: build at n = 131072 (596.1 MB / 1,048,576 units; traffic is proportional to
# units), scan at n = 1,048,576 and B = 48 (58.5 MB read + 81.9 MB written = 140.4 MB / 8,388,608 units; part of the
# score writes is still in L2 when the kernel ends), the three top-k kernels at n = 1,048,576, k = 4096 (8.4 + 134.25 +
# 2.2 MB read, 3.7 MB written / 8,388,608 units; valid for the single-pass path only), attention at k = 4096 (66.1 MB read + 1.05 MB
# written; proportional to k, not to n: 67.1 MB / (32 heads x 4096 rows) = 512.3 B per selected row).
# Multiplied by the units of a launch in the JSON line.
NCU_TRAFFIC_BYTES_PER_TOKEN_KVHEAD = {"build_planes_kernel": 568.5, "scan_kernel": 16.74, "topk_*": 17.7}
NCU_TRAFFIC_BYTES_PER_SELECTED_ROW = 512.3
NCU_SCAN_WARP_INSTRUCTIONS_PER_BLOCK_OF_48_ROWS = 222.7         # smsp__inst_executed.sum / (n * Hkv / 64) at B = 48 (profiles/scan_kernel_n1M_B48.md)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps (default: 1000 decode steps of ~0.12 ms; 3 for --impl reference, whose steps take seconds)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--n", type=int, default=WORKLOAD["n"], help="tokens per session (default: the 1M configuration)")
    ap.add_argument("--budget", type=int, default=WORKLOAD["B"])
    ap.add_argument("--k", type=int, default=WORKLOAD["k"])
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-host-resident", action="store_true", help="skip the pinned-host-planes scan leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-session-kernels", action="store_true", help="skip the once-per-session statistics / rotation kernels")
    ap.add_argument("--cpu-sample-tokens", type=int, default=262144)
    ap.add_argument("--ref-sample-tokens", type=int, default=65536)
    ap.add_argument("--config4", action="store_true",
                    help="instead of the default line: the 16-session agentic batch (planes in pinned host memory), "
                         "one decode step over --layers independently seeded layers")
    ap.add_argument("--config5", action="store_true",
                    help="the budget sweep at n = 1M (water-filled budgets and fixed top-r channels) instead of the default step")
    ap.add_argument("--plan-layers", action="store_true",
                    help="per-layer budgets: measure every layer's error at every level, plan at mean --budget, re-run; use with "
                         "--layers L --n N")
    ap.add_argument("--layers", type=int, default=None, help="config 4: layers timed (default 36); --plan-layers: synthetic layers (default 12)")
    ap.add_argument("--lanes", type=int, default=4, help="config 4: stream lanes over which the sessions are spread")
    ap.add_argument("--stage", choices=STAGES, help="time ONE stage on small synthetic buffers instead of the bench (for profilers)")
    ap.add_argument("--iters", type=int, default=10, help="--stage: timed samples")
    ap.add_argument("--repeat", type=int, default=1, help="--stage: launches per timed sample (back to back; the event timer resolves ~2 us)")
    ap.add_argument("--kv-heads", type=int, default=WORKLOAD["Hkv"], help="--stage only")
    ap.add_argument("--q-heads", type=int, default=WORKLOAD["Hq"], help="--stage only")
    ap.add_argument("--heads-per-plan", dest="heads_per_plan_arg", type=int, default=WORKLOAD["heads_per_plan"], help="--stage only")
    ap.add_argument("--host-planes", action="store_true", help="--stage scan: planes and scales in pinned host memory")
    ap.add_argument("--host-rows", action="store_true", help="--stage union: K/V rows in pinned host memory")
    ap.add_argument("--ctas", type=int, default=0, help="--stage: CTAs per plan of the scan (0 = automatic)")
    ap.add_argument("--no-flush", action="store_true", help="--stage: do not write a 256 MB buffer between iterations")
    a = ap.parse_args()
    if a.steps is None:
        a.steps = 3 if a.impl == "reference" else 1000
    return a


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy bandwidth)"
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons through NVML (read-only) from a thread while the timed region runs."""

    def __init__(self, gpu_index: int, period_s: float = 0.002):
        import threading
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            # NVML indexes physical devices: map through CUDA_VISIBLE_DEVICES when it lists indices
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            ids = [v for v in vis.split(",") if v.strip().isdigit()]
            phys = int(ids[gpu_index]) if gpu_index < len(ids) else gpu_index
            self._h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as e:                                  # no NVML: report that, never guess
            self._nv = None
            self.err = repr(e)
            return
        self._period = period_s
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def _run(self):
        nv = self._nv
        names = [("hw_slowdown", nv.nvmlClocksEventReasonHwSlowdown if hasattr(nv, "nvmlClocksEventReasonHwSlowdown") else 0x8),
                 ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4)]
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                r = int(get_reasons(self._h))
                for nm, bit in names:
                    if r & bit:
                        self.reasons.add(nm)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
            except Exception:
                pass
            time.sleep(self._period)

    def mark(self):
        """The timed region starts here (samples before it belong to the warm-up steps, which run the same kernels)."""
        self.marked = len(self.samples)

    def in_region(self):
        return len(self.samples) - getattr(self, "marked", 0) if self._nv is not None else 1 << 30

    def stop(self):
        if self._nv is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable: " + self.err]}
        self._stop.set()
        self._thread.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "sm_mhz_min": min(self.samples) if self.samples else None,
                "power_w_max": max(self.power) if self.power else None, "samples": len(self.samples),
                "samples_in_timed_region": len(self.samples) - getattr(self, "marked", 0),
                "reasons": sorted(self.reasons)}


def bits_per_token(depth_row) -> float:
    t = np.asarray(depth_row).astype(np.int64)
    return float(t.sum()) + float((t > 0).sum()) * 16.0 / 64.0


# ------------------------------------------------------------------------------------------------ ours
def run_ours(args):
    from paper_2609_17652_b200 import binding as fb
    from workloads.synth import make_layer

    rank, world, local_rank = fdist.init_from_env(args.gpus, backend="nccl")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    n, Hkv, Hq, d = args.n, WORKLOAD["Hkv"], WORKLOAD["Hq"], WORKLOAD["d"]
    B, k, hpp = args.budget, args.k, WORKLOAD["heads_per_plan"]
    G = Hq // Hkv

    # weak scaling: every rank owns one independent session (its own seed); no data-path collective.
    # The session has N_LAYERS independently seeded layers' stores; consecutive steps take consecutive layers, as the
    # decode step of a model does, so no plane byte of a step is still in L2 from the step before (4 x 58 MB > 126 MB).
    session = fdist.sessions_of_rank(rank, world, n_sessions=world)[0]
    lay = fb.make_layout(Hkv, Hq, n, d)
    ctx = fb.Context(local_rank, fb.fathom_scratch_bytes(lay, k))
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    layers = []
    build_ts = []
    for li in range(N_LAYERS):
        Ll = make_layer(n, Hkv, Hq, d, seed=2, session=session, layer=li, device=str(dev), want_rows=(li == 0))
        pl = torch.zeros((Hkv, d, 4, lay.plane_stride_words), dtype=torch.int64, device=dev)
        sc = torch.zeros((Hkv, d, lay.scale_stride), dtype=torch.int16, device=dev)
        for it in range(4 if li == 0 else 3):                    # once per sequence: timed here, L2 flushed, not part of the step
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); ctx.fathom_build_planes(lay, Ll.K, pl, sc, stream); b.record(stream)
            torch.cuda.synchronize()
            if it or li:
                build_ts.append(a.elapsed_time(b) * 1e3)
        if li == 0:
            L = Ll
        layers.append({"planes": pl, "scales": sc, "q": Ll.q, "var": Ll.var})
        if li:
            del Ll
    build_us = statistics.median(build_ts)
    planes, scales = layers[0]["planes"], layers[0]["scales"]
    depth = torch.zeros((Hq // hpp, d), dtype=torch.uint8, device=dev)
    scores = torch.zeros((Hq, lay.score_stride), dtype=torch.float32, device=dev)
    idx = torch.zeros((Hq, k), dtype=torch.int32, device=dev)
    out = torch.zeros((Hq, d), dtype=torch.float32, device=dev)
    sm_scale = 1.0 / math.sqrt(d)

    stage_names = ["alloc_depth", "scan", "topk", "sparse_attend"]
    topk_passes = fb.fathom_topk_passes(lay, k)                 # 1: sampled estimate + one collection pass; 2: histogram + filter
    # single pass: sample histogram, collection, selection (3 kernels); two passes: histogram, filter, select, emit (4)
    launches_per_step = {"alloc_depth": 1, "scan": 1, "topk": 3 if topk_passes == 1 else 4, "sparse_attend": 1}

    def stage(i, W, st, q=None, var=None, result=None):
        """Stage i of the decode step on layer store W: alloc_depth, scan, topk, sparse_attend (`result`: where the
        attention output goes instead of the device buffer `out`)."""
        q = W["q"] if q is None else q
        var = W["var"] if var is None else var
        if i == 0:
            ctx.fathom_alloc_depth(lay, q, var, fb.DEPTH_WATERFILL, B, hpp, depth, st)
        elif i == 1:
            ctx.fathom_scan(lay, W["planes"], W["scales"], q, depth, hpp, scores, st)
        elif i == 2:
            ctx.fathom_topk(lay, scores, k, 0, 0, idx, st)
        else:
            ctx.fathom_sparse_attend(lay, q, L.Krows, L.Vrows, idx, k, sm_scale, out if result is None else result, st)

    def step(s, events=None):
        W = layers[s % N_LAYERS]
        for i in range(4):
            if events is not None:
                events[i].record(stream)
            stage(i, W, stream)
        if events is not None:
            events[4].record(stream)

    sampler = ClockSampler(local_rank, period_s=0.0005) if rank == 0 else None   # samples from the warm-up steps on: same load
    for s in range(max(args.warmup, 3)):
        step(s)
    torch.cuda.synchronize()

    # ---- timed region: exactly `steps` decode steps between two CUDA events on the launching stream, clocks sampled
    #      meanwhile.  No event is recorded inside it: an event between two launches would cut the programmatic dependent
    #      launches that let a kernel become resident while its predecessor drains.
    fdist.barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.mark()
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall = time.perf_counter()
    e_begin.record(stream)
    for s in range(args.steps):
        step(s)
    e_end.record(stream)
    torch.cuda.synchronize()
    t_wall = time.perf_counter() - t_wall
    fdist.barrier()
    replay_ms = 0.0
    if sampler and sampler.in_region() < 3:
        # the region was shorter than a few NVML queries: the same steps go on, untimed, until the clocks under this very
        # load have been read a few times (at most ~0.5 s)
        t0 = time.perf_counter()
        while sampler.in_region() < 3 and time.perf_counter() - t0 < 0.5:
            for s in range(args.steps):
                step(s)
            torch.cuda.synchronize()
        replay_ms = (time.perf_counter() - t0) * 1e3
    clocks = sampler.stop() if sampler else None
    if clocks is not None:
        clocks["sampled_over"] = "the timed region" if replay_ms == 0.0 else (
            f"the timed region and an untimed continuation of the same steps for {replay_ms:.0f} ms (the region alone was "
            "shorter than three NVML reads)")
    total_ms = fdist.max_over_ranks(e_begin.elapsed_time(e_end))
    ms_per_step = total_ms / args.steps
    # ---- the same `steps` steps once more with an event between the stages: the per-stage times (and the roofline's
    #      kernel duration) come from this pass; its stages do not overlap, so they add up to slightly more than a step
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    for s in range(args.steps):
        step(s, ev[s])
    torch.cuda.synchronize()
    stage_us = {nm: 1e3 * statistics.mean(ev[s][i].elapsed_time(ev[s][i + 1]) for s in range(args.steps))
                for i, nm in enumerate(stage_names)}
    staged_step_us = 1e3 * ev[0][0].elapsed_time(ev[-1][4]) / args.steps
    stage_us["build_planes"] = build_us
    status = ctx.fathom_device_status()
    step(0)                                                     # depth, scores, idx of layer 0 for the legs below
    torch.cuda.synchronize()

    # per launch, all plans: a plan's rows are read once by the CTAs that serve it (twice for plans of eight heads, which two
    # groups of four heads share); mean over the layers the steps rotate over (their plans differ slightly)
    per_layer_bytes, per_layer_bits = [], []
    for W in reversed(layers):                                  # layer 0 last: its depths stay in `depth`
        stage(0, W, stream)
        torch.cuda.synchronize()
        dh = depth.cpu().numpy()
        per_layer_bytes.append(sum(bits_per_token(r) for r in dh) / 8.0 * n * max(1, hpp // 4))
        per_layer_bits.append(float(np.mean([bits_per_token(r) for r in dh])))
    depth_h = depth.cpu().numpy()
    bits = float(np.mean(per_layer_bits))
    plane_bytes_read = float(np.mean(per_layer_bytes))
    alg_bytes = {
        "build_planes": n * Hkv * (d * 4 + 68.0),
        "scan": plane_bytes_read + 4.0 * Hq * n,
        "topk": topk_passes * 4.0 * Hq * n,
        "sparse_attend": Hq * k * d * 2 * 2.0,
    }
    peak, peak_src = measured_peaks()

    def roof(stage_key, t_us, kernel, unit_count):
        ach = alg_bytes[stage_key] / (t_us * 1e-6) / 1e9
        tr = NCU_TRAFFIC_BYTES_PER_TOKEN_KVHEAD.get(kernel)
        return {"kernel": kernel, "bound": "hbm", "achieved": round(ach, 1), "peak": peak, "unit": "GB/s",
                "frac": round(ach / peak, 4),
                "traffic": (NCU_TRAFFIC_BYTES_PER_SELECTED_ROW * Hq * k if kernel == "attend_*" else
                            (tr * unit_count if tr and not (kernel == "topk_*" and topk_passes != 1) else None)),
                "algorithmic_bytes": alg_bytes[stage_key], "launch_us": round(t_us, 2), "peak_source": peak_src}

    # ---- isolated stage timings with an L2 flush before every launch (cold-cache view of each stage)
    iso_us = {"build_planes": build_us}
    for i, nm in enumerate(stage_names):
        ts = []
        for _ in range(10):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); stage(i, layers[0], stream); b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) * 1e3)
        iso_us[nm] = statistics.median(ts)

    result = {
        "metric": METRIC, "value": None, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u64 bit planes + f32 accumulate", "data": "synthetic",
        "config": {"workload": WORKLOAD["name"], "n": n, "kv_heads": Hkv, "q_heads": Hq, "d": d, "budget_bits": B,
                   "k": k, "heads_per_plan": hpp, "sessions_per_gpu": 1, "parallelism": f"{world} independent session(s), one per GPU",
                   "step": "one decode step of one layer: fathom_alloc_depth -> fathom_scan -> fathom_topk -> fathom_sparse_attend; "
                           "fathom_build_planes runs once per sequence and is timed separately (once_per_sequence)",
                   "l2": f"consecutive steps take the stores of {N_LAYERS} independently seeded layers in turn ({N_LAYERS} x 58 MB of plane "
                         "rows read, 134 MB of scores written and re-read, 67 MB of rows gathered from 4 GiB per step): nothing a step "
                         "reads is left in the 126 MB L2 by the step before; no explicit flush in the timed region"},
    }
    keys_per_step = n * Hkv * world
    result["value"] = keys_per_step / (ms_per_step * 1e-3)
    result["gpu_launches"] = args.steps * sum(launches_per_step.values())
    result["clocks"] = clocks
    result["stage_us"] = {k_: round(v, 2) for k_, v in stage_us.items()}
    result["stage_us_isolated_l2_flushed"] = {k_: round(v, 2) for k_, v in iso_us.items()}
    result["decode_step_us_per_layer"] = round(1e3 * ms_per_step, 2)
    result["decode_step_us_per_layer_with_stage_events"] = round(staged_step_us, 2)
    result["once_per_sequence"] = {"build_planes_us": round(build_us, 2), "keys_per_s": n * Hkv / (build_us * 1e-6),
                                   "step_with_build_ms": round(ms_per_step + build_us * 1e-3, 4),
                                   "keys_per_s_step_with_build": keys_per_step / (ms_per_step * 1e-3 + build_us * 1e-6)}
    result["bits_per_token"] = round(bits, 2)
    result["scan"] = {
        "keys_per_s": n * Hkv / (stage_us["scan"] * 1e-6),
        "plane_and_scale_bytes_read": plane_bytes_read,
        "gbs_index_bytes_only": round(plane_bytes_read / (stage_us["scan"] * 1e-6) / 1e9, 1),
        "gbs_with_score_writes": round(alg_bytes["scan"] / (stage_us["scan"] * 1e-6) / 1e9, 1),
    }
    # ---- the scan kernel without launch gaps: 40 launches in a row between two events, over the four layers in turn (each
    #      launch reads another layer's 58 MB of plane rows, 233 MB in all: what a launch reads was evicted since its last use)
    depth_l = []
    for W in layers:
        d_l = torch.zeros_like(depth)
        ctx.fathom_alloc_depth(lay, W["q"], W["var"], fb.DEPTH_WATERFILL, B, hpp, d_l, stream)
        depth_l.append(d_l)
    for rep in range(2):                                        # the first round warms up
        a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a_.record(stream)
        for it in range(40):
            W = layers[it % N_LAYERS]
            ctx.fathom_scan(lay, W["planes"], W["scales"], W["q"], depth_l[it % N_LAYERS], hpp, scores, stream)
        b_.record(stream)
        torch.cuda.synchronize()
    scan_b2b_us = a_.elapsed_time(b_) * 1e3 / 40
    result["scan"]["us_back_to_back_over_the_layers"] = round(scan_b2b_us, 2)
    result["scan"]["gbs_with_score_writes_back_to_back"] = round(alg_bytes["scan"] / (scan_b2b_us * 1e-6) / 1e9, 1)
    # ---- the top-k chain (sample, collection, selection) without launch gaps: 40 calls in a row on the scores of the last scan
    for rep in range(2):
        a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a_.record(stream)
        for it in range(40):
            ctx.fathom_topk(lay, scores, k, 0, 0, idx, stream)
        b_.record(stream)
        torch.cuda.synchronize()
    topk_b2b_us = a_.elapsed_time(b_) * 1e3 / 40
    result["topk"] = {"us_in_the_step_between_events": round(stage_us["topk"], 2), "us_back_to_back": round(topk_b2b_us, 2),
                      "score_bytes": alg_bytes["topk"], "gbs_back_to_back": round(alg_bytes["topk"] / (topk_b2b_us * 1e-6) / 1e9, 1)}
    # ---- the configuration's second budget (B = 80) through the same kernels: bytes read, scan time
    other = {}
    for B2 in (80,):
        d2 = torch.zeros_like(depth)
        ctx.fathom_alloc_depth(lay, L.q, L.var, fb.DEPTH_WATERFILL, B2, hpp, d2, stream)
        ts = []
        for it in range(13):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); ctx.fathom_scan(lay, planes, scales, L.q, d2, hpp, scores, stream); b.record(stream)
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(a.elapsed_time(b) * 1e3)
        d2h = d2.cpu().numpy()
        rd = sum(bits_per_token(r) for r in d2h) / 8.0 * n * max(1, hpp // 4)
        t2 = statistics.median(ts)
        other[str(B2)] = {"bits_per_token": round(float(np.mean([bits_per_token(r) for r in d2h])), 2), "scan_us_l2_flushed": round(t2, 2),
                          "plane_and_scale_bytes_read": rd, "gbs_index_bytes_only": round(rd / (t2 * 1e-6) / 1e9, 1),
                          "gbs_with_score_writes": round((rd + 4.0 * Hq * n) / (t2 * 1e-6) / 1e9, 1)}
    # ---- one plan per query head instead of one per KV group (the paper shares a plan among the G heads of a group: the
    #      planes are then read once for all of them, and the bit test of a token and row serves G adds instead of one)
    if hpp != 1:
        d1 = torch.zeros((Hq, d), dtype=torch.uint8, device=dev)
        ctx.fathom_alloc_depth(lay, L.q, L.var, fb.DEPTH_WATERFILL, B, 1, d1, stream)
        ts = []
        for it in range(13):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); ctx.fathom_scan(lay, planes, scales, L.q, d1, 1, scores, stream); b.record(stream)
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(a.elapsed_time(b) * 1e3)
        rd = sum(bits_per_token(r) for r in d1.cpu().numpy()) / 8.0 * n
        t1 = statistics.median(ts)
        result["scan_per_query_head_plans"] = {"heads_per_plan": 1, "scan_us_l2_flushed": round(t1, 2), "plane_and_scale_bytes_read": rd,
                                               "gbs_index_bytes_only": round(rd / (t1 * 1e-6) / 1e9, 1),
                                               "gbs_with_score_writes": round((rd + 4.0 * Hq * n) / (t1 * 1e-6) / 1e9, 1)}
    stage(1, layers[0], stream); stage(2, layers[0], stream)      # scores and picks of the default budget again
    result["scan_other_budgets"] = other
    # the headline roofline is the scan kernel's: the kernel the metric and the targets are written for
    scan_s = stage_us["scan"] * 1e-6
    result["roofline"] = roof("scan", stage_us["scan"], "scan_kernel", n * Hkv)
    result["roofline"]["frac_index_bytes_only"] = round(plane_bytes_read / scan_s / 1e9 / peak, 4)
    # what two events around ONE launch cost by themselves: a one-element fill kernel between two events
    tiny = torch.zeros(1, device=dev)
    ov = []
    for _ in range(50):
        a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a_.record(stream); tiny.fill_(1.0); b_.record(stream)
        torch.cuda.synchronize()
        ov.append(a_.elapsed_time(b_) * 1e3)
    result["roofline"]["event_bracket_overhead_us"] = round(statistics.median(ov), 2)
    result["roofline"]["launch_us_back_to_back"] = round(scan_b2b_us, 2)
    result["roofline"]["frac_back_to_back"] = round(alg_bytes["scan"] / (scan_b2b_us * 1e-6) / 1e9 / peak, 4)
    result["roofline"]["note_back_to_back"] = ("launch_us is the stage time inside the decode step (an event on either side of the call: it "
                                               "includes the launch latency the events expose - event_bracket_overhead_us is what a one-element "
                                               "fill kernel measures between two events); launch_us_back_to_back is the mean of 40 launches "
                                               "in a row over the four layers' stores in turn (no gaps; every launch reads rows evicted since their last use)")
    result["roofline"]["note"] = ("algorithmic bytes = plane words and scales read + fp32 scores written; frac_index_bytes_only counts the "
                                  "plane words and scales alone (the paper's GB/s convention); with the scores materialised that figure "
                                  "cannot exceed bytes_read / (bytes_read + bytes_written) = %.2f" % (plane_bytes_read / alg_bytes["scan"]))
    result["roofline_other_kernels"] = {
        "build_planes (once per sequence)": roof("build_planes", build_us, "build_planes_kernel", n * Hkv),
        f"topk ({topk_passes} pass{'es' if topk_passes > 1 else ''} over the scores)": roof("topk", stage_us["topk"], "topk_*", n * Hkv),
        "sparse_attend": roof("sparse_attend", stage_us["sparse_attend"], "attend_*", n * Hkv),
    }
    # the scan's arithmetic: one tensor-core multiply-add per (token, active row, head part) and, on the CUDA cores, the
    # expansion of every plane bit into a signed fp16 operand (one shift + one logic op per pair of elements)
    elements = float(n) * sum(int(r.sum()) for r in depth_h)                 # (token, active row) pairs of one launch, all plans
    issue_peak = 148 * 4 * 1.965e9                              # warp instructions per second (four schedulers per SM)
    result["roofline"]["alt_bound"] = {
        "bound": "alu", "unit": "G warp instructions/s", "peak": round(issue_peak / 1e9, 1),
        "achieved": round(elements / 3072.0 * NCU_SCAN_WARP_INSTRUCTIONS_PER_BLOCK_OF_48_ROWS / scan_s / 1e9, 1),
        "frac": round(elements / 3072.0 * NCU_SCAN_WARP_INSTRUCTIONS_PER_BLOCK_OF_48_ROWS / scan_s / issue_peak, 4),
        "note": "issue-slot view: warp instructions per 64 tokens x 48 rows from the committed ncu summary (profiles/), scaled by the "
                "launch's (token, row) pairs; peak = 148 SMs x 4 schedulers x 1.965 GHz"}
    result["targets"] = {
        "hbm_resident_scan_frac_of_hbm_peak": {"target": 0.70, "achieved_with_score_writes": result["roofline"]["frac"],
                                               "achieved_index_bytes_only": result["roofline"]["frac_index_bytes_only"],
                                               "met": bool(result["roofline"]["frac"] >= 0.70)},
    }

    # ---- attention gathers 256-byte rows scattered over 2 + 2 GiB: every row opens a DRAM page, so the copy peak is not
    #      the bound that matters.  A micro-benchmark of a pure gather (half a warp per row, 8 loads in flight, rows
    #      summed and dropped) on this machine's B200 read 262,144 such rows (as many as k = 4096 x 32 heads x {K, V}) in
    #      22.5 us (2.98 TB/s) and 1,048,576 rows at 4.68 TB/s.
    if Hq * k * 2 == 262144:
        result["roofline_other_kernels"]["sparse_attend"]["alt_bound"] = {
            "bound": "scattered 256-byte row gather", "pure_gather_us": 22.5, "attend_us": round(stage_us["sparse_attend"], 2),
            "frac": round(22.5 / stage_us["sparse_attend"], 3),
            "note": "pure-gather time measured once by a micro-benchmark (same row count and row size, L2 flushed)"}

    # ---- the decode part of the step (everything but the one-off build) replayed as one CUDA graph: ten replays back
    #      to back per sample (a single replay would include the idle time before the graph launch arrives), median of 10
    graph_us = None
    try:
        gs = torch.cuda.Stream()
        gs.wait_stream(stream)
        with torch.cuda.stream(gs):
            for W in layers:
                for i in range(4):
                    stage(i, W, gs)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=gs):
                for W in layers:                                    # one graph = the decode steps of N_LAYERS layers
                    for i in range(4):
                        stage(i, W, gs)
        torch.cuda.synchronize()
        ts = []
        for it in range(13):                                        # three replays back to back per sample, as the layers
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)   # of a model would follow each other
            a.record(stream)
            for _ in range(3):
                g.replay()
            b.record(stream)
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(a.elapsed_time(b) * 1e3 / (3.0 * N_LAYERS))
        graph_us = round(statistics.median(ts), 2)
        del g
    except Exception as e:                                      # report, never hide
        graph_us = "capture failed: " + repr(e)
    result["decode_step_us_per_layer_cuda_graph"] = graph_us

    # ---- the same decode step with scan and selection fused (scores never written): alloc, scan_topk, attend
    def fused_on(W, st):
        ctx.fathom_alloc_depth(lay, W["q"], W["var"], fb.DEPTH_WATERFILL, B, hpp, depth, st)
        ctx.fathom_scan_topk(lay, W["planes"], W["scales"], W["q"], depth, hpp, k, 0, 0, idx, st)
        ctx.fathom_sparse_attend(lay, W["q"], L.Krows, L.Vrows, idx, k, sm_scale, out, st)
    for s_ in range(3):
        fused_on(layers[s_ % N_LAYERS], stream)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for s_ in range(args.steps):
        fused_on(layers[s_ % N_LAYERS], stream)
    b.record(stream)
    torch.cuda.synchronize()
    result["decode_step_fused_us_per_layer"] = round(a.elapsed_time(b) * 1e3 / args.steps, 2)
    stage(0, layers[0], stream); stage(1, layers[0], stream); stage(2, layers[0], stream)   # layer 0's depths, scores, picks again
    result["device_status"] = status
    result["wall_ms_per_step"] = round(1e3 * t_wall / args.steps, 4)

    # ---- planes in pinned host memory, read zero-copy by the scan kernel over the host link
    if rank == 0 and not args.no_host_resident:
        result["host_resident_scan"] = host_resident_leg(ctx, lay, planes, scales, L, depth, hpp, scores, stream, per_layer_bytes[-1])
        result["host_resident_row_fetch"] = row_fetch_leg(ctx, lay, L, idx, k, G, stream,
                                                          result["host_resident_scan"]["link_peak_gbs"])
        result["targets"]["host_resident_scan_frac_of_measured_link"] = {
            "target": 0.80, "achieved": result["host_resident_scan"]["frac_of_measured_link"],
            "met": bool(result["host_resident_scan"]["frac_of_measured_link"] >= 0.80)}

    # ---- once-per-session kernels of the raw and the KLT-rotated store (not part of the step): statistics, rotation
    if rank == 0 and not args.no_session_kernels:
        result["session_kernels"] = session_kernels_leg(ctx, lay, L, stream, peak)

    # ---- end to end through the C ABI from HOST buffers: H2D of the step's inputs and D2H of its result are timed
    if not args.no_e2e:
        result["e2e"] = e2e_leg(args, layers, stage, out, stream, keys_per_step)
    else:
        result["e2e"] = None

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(args.cpu_sample_tokens, B, min(k, 2048), hpp)
    fdist.barrier()
    if rank == 0:
        print(json.dumps(result))
    ctx.close()
    fdist.shutdown()


def session_kernels_leg(ctx, lay, L, stream, hbm_peak):
    """Times fathom_channel_variance, fathom_calibrate and fathom_rotate_keys on the bench's keys (L2 flushed before
    each launch) and reports them against the HBM peak and, for the two contractions, the tf32 tensor peak
    (measured bf16 peak x the nominal tf32 : bf16 ratio 1.1 : 2.25)."""
    Hkv, n, d = L.K.shape
    dev = L.K.device
    mean = torch.zeros((Hkv, d), device=dev); var = torch.zeros((Hkv, d), device=dev)
    cov = torch.zeros((Hkv, d, d), device=dev)
    basis = torch.linalg.qr(torch.randn(Hkv, d, d, device=dev))[0].contiguous()
    K_rot = torch.empty((Hkv, n, d), device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    calls = {
        "channel_variance": lambda: ctx.fathom_channel_variance(lay, L.K, mean, var, stream),
        "calibrate": lambda: ctx.fathom_calibrate(lay, L.K, mean, cov, stream),
        "rotate_keys": lambda: ctx.fathom_rotate_keys(lay, L.K, mean, basis, K_rot, stream),
    }
    kbytes = float(L.K.numel() * L.K.element_size())
    alg_bytes = {"channel_variance": kbytes, "calibrate": kbytes, "rotate_keys": kbytes + 4.0 * K_rot.numel()}
    products = {"calibrate": 2, "rotate_keys": 3}                  # tf32 products per multiply of the split operands
    tf32_peak = None
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            tf32_peak = float(json.load(f)["bf16_tflops"]) * 1.1 / 2.25
    out = {}
    for nm, fn in calls.items():
        ts = []
        for it in range(8):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream)
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(a.elapsed_time(b) * 1e3)
        t_us = statistics.median(ts)
        gbs = alg_bytes[nm] / (t_us * 1e-6) / 1e9
        r = {"us": round(t_us, 1), "algorithmic_bytes": alg_bytes[nm], "achieved_gbs": round(gbs, 1), "frac_of_hbm_peak": round(gbs / hbm_peak, 4)}
        if nm in products:
            tf = products[nm] * 2.0 * n * Hkv * d * d / (t_us * 1e-6) / 1e12
            r.update({"tensor_tflops_tf32": round(tf, 1), "tf32_peak_tflops": round(tf32_peak, 1) if tf32_peak else None,
                      "frac_of_tf32_peak": round(tf / tf32_peak, 4) if tf32_peak else None})
        out[nm] = r
    out["note"] = ("once per session, not in the timed step; calibrate reads the keys once (covariance and sums of keys centred "
                   "on a shift); the contractions run as tcgen05.mma on tf32 operands split in head and tail")
    return out


def host_resident_leg(ctx, lay, planes, scales, L, depth, hpp, scores, stream, plane_bytes_read):
    hp = torch.empty(planes.shape, dtype=planes.dtype, pin_memory=True); hp.copy_(planes)
    hs = torch.empty(scales.shape, dtype=scales.dtype, pin_memory=True); hs.copy_(scales)
    # host-link probe: one pinned -> device copy of 1 GiB, best of 10
    src = torch.empty(1 << 30, dtype=torch.uint8, pin_memory=True)
    dst = torch.empty(1 << 30, dtype=torch.uint8, device=planes.device)
    best = 1e9
    for _ in range(10):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream); dst.copy_(src, non_blocking=True); b.record(stream)
        torch.cuda.synchronize()
        best = min(best, a.elapsed_time(b))
    link_gbs = (1 << 30) / (best * 1e-3) / 1e9
    ts = []
    for it in range(8):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        ctx.fathom_scan(lay, hp, hs, L.q, depth, hpp, scores, stream)
        b.record(stream)
        torch.cuda.synchronize()
        if it >= 3:
            ts.append(a.elapsed_time(b))
    t = statistics.median(ts)
    gbs = plane_bytes_read / (t * 1e-3) / 1e9
    del src, dst
    return {"scan_ms": round(t, 4), "bytes_over_link": plane_bytes_read, "gbs": round(gbs, 2),
            "link_peak_gbs": round(link_gbs, 2), "frac_of_measured_link": round(gbs / link_gbs, 4),
            "link_probe": "1 GiB pinned->device copy, best of 10"}


def row_fetch_leg(ctx, lay, L, idx, k, G, stream, link_gbs):
    """K/V rows in pinned host memory: the union of each group's winners is fetched once over the host link."""
    hK = torch.empty(L.Krows.shape, dtype=L.Krows.dtype, pin_memory=True); hK.copy_(L.Krows)
    hV = torch.empty(L.Vrows.shape, dtype=L.Vrows.dtype, pin_memory=True); hV.copy_(L.Vrows)
    dev = L.Krows.device
    Kst = torch.empty((L.Hkv, G * k, L.d), dtype=L.Krows.dtype, device=dev)
    Vst = torch.empty_like(Kst)
    loc = torch.empty((L.Hq, k), dtype=torch.int32, device=dev)
    cnt = torch.zeros((L.Hkv,), dtype=torch.int32, device=dev)
    ts = []
    for it in range(8):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        ctx.fathom_gather_union(lay, idx, k, hK, hV, Kst, Vst, loc, cnt, stream)
        b.record(stream)
        torch.cuda.synchronize()
        if it >= 3:
            ts.append(a.elapsed_time(b))
    t = statistics.median(ts)
    rows = int(cnt.sum().item())
    nbytes = rows * L.d * 2 * L.Krows.element_size()
    gbs = nbytes / (t * 1e-3) / 1e9
    del hK, hV
    return {"ms": round(t, 4), "distinct_rows": rows, "picks": int(L.Hq * k), "bytes_over_link": nbytes,
            "gbs": round(gbs, 2), "frac_of_measured_link": round(gbs / link_gbs, 4)}


def e2e_leg(args, layers, stage, out, stream, keys_per_step):
    """The decode step end to end from HOST buffers: what a decode step ships is the layer's query and channel statistics
    in (pinned host memory -> device, inside the timed region, every step) and the attention output back (device ->
    pinned host); the store and the K/V rows are resident, as they are between the steps of a session."""
    # q and var of a step sit side by side in one pinned staging buffer and cross in one copy
    nq, nv = layers[0]["q"].numel(), layers[0]["var"].numel()
    hqv = [torch.empty(nq + nv, dtype=torch.float32, pin_memory=True) for _ in layers]
    for W, h in zip(layers, hqv):
        h[:nq].copy_(W["q"].reshape(-1)); h[nq:].copy_(W["var"].reshape(-1))
    hout = torch.empty(out.shape, dtype=out.dtype, pin_memory=True)
    dqv = torch.empty(nq + nv, dtype=torch.float32, device=out.device)
    dq, dvar = dqv[:nq].view(layers[0]["q"].shape), dqv[nq:].view(layers[0]["var"].shape)
    h2d = hqv[0].numel() * hqv[0].element_size()
    d2h = hout.numel() * hout.element_size()
    # The attention kernel writes its 16 KB straight into the pinned host buffer (a device-accessible pointer like any other
    # to the C ABI): 126.5 us per step against 129.4 us with a device buffer and a copy (FATHOM_BENCH_E2E_DIRECT_OUT=0).  The
    # inputs do need their copy: with q and var left in pinned host memory every CTA of the scan reads them over the link
    # (167 us per step).
    direct_out = os.environ.get("FATHOM_BENCH_E2E_DIRECT_OUT", "1") != "0"

    def e2e_step(s):
        li = s % len(layers)
        dqv.copy_(hqv[li], non_blocking=True)
        for i in range(4):
            stage(i, layers[li], stream, q=dq, var=dvar, result=hout if direct_out else None)
        if not direct_out:
            hout.copy_(out, non_blocking=True)

    steps = args.steps
    for s in range(3):
        e2e_step(s)
    torch.cuda.synchronize()
    fdist.barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for s in range(steps):
        e2e_step(s)
    b.record(stream)
    torch.cuda.synchronize()
    ms = fdist.max_over_ranks(a.elapsed_time(b)) / steps
    # what arrived in host memory is what the same step leaves in the device buffer
    li = (steps - 1) % len(layers)
    for i in range(4):
        stage(i, layers[li], stream, q=dq, var=dvar)
    torch.cuda.synchronize()
    if not torch.equal(hout, out.cpu()):
        raise RuntimeError("end-to-end leg: the attention output in host memory differs from the device-resident step's")
    return {"value": keys_per_step / (ms * 1e-3), "unit": UNIT, "ms_per_step": round(ms, 4), "steps": steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "what": "per step: q [32][128] and var [8][128] (fp32, one pinned staging buffer, one copy) from the host to the device, the four C-ABI calls "
                    "of the decode step on the resident store and rows, out [32][128] " +
                    ("written by the attention kernel straight into pinned host memory" if direct_out else "copied back to pinned host memory")}


# ------------------------------------------------------------------------------------------------ config 4
class Config4:
    """Agentic multi-session batch (config 4): 16 concurrent sessions, n log-uniform in [65536, 1048576] (ragged, not
    multiples of 64), Qwen3-8B layer shape, B = 48, k = 2048.  As in the paper's offload harness (Sec. 4) the planes, the
    scales AND the K/V rows of every session live in pinned host memory.  One decode step of a layer = for every session:
    alloc_depth -> scan (planes read over the host link; the sessions of a group in one fathom_scan_batch launch) ->
    top-k -> union of each group's winners fetched once from the host rows (fathom_gather_union) -> attention over the
    staged rows.  The scans run on the main stream; top-k, row fetch and attention of a session run on one of `lanes` side
    streams, so the link carries the next group's planes while the previous group's rows and selection are worked on.
    Layers are independently seeded and processed one at a time with reused buffers (36 layers of planes and rows would be
    1.1 TB of pinned memory): build_layer() refills the host stores (untimed), decode_layer() enqueues the step."""

    def __init__(self, fb, dev, lanes=4, n_sessions=16, lo=65536, hi=1048576, k=2048, budget=48, host_rows=True):
        from workloads.synth import session_lengths
        self.fb, self.dev = fb, dev
        self.Hkv, self.Hq, self.d, self.B, self.k, self.hpp = 8, 32, 128, budget, k, 4
        self.G = self.Hq // self.Hkv
        Hkv, Hq, d = self.Hkv, self.Hq, self.d
        self.lengths = session_lengths(n_sessions, lo, hi, seed=0)
        nmax = max(self.lengths)
        self.lay_max = fb.make_layout(Hkv, Hq, nmax, d)
        self.lay_stage = fb.make_layout(Hkv, Hq, self.G * k, d)
        self.main = torch.cuda.current_stream()
        self.ctx = fb.Context(dev.index or 0, fb.fathom_scratch_bytes(self.lay_max, k))
        self.lanes = []
        for _ in range(max(1, lanes)):
            self.lanes.append({"ctx": fb.Context(dev.index or 0, fb.fathom_scratch_bytes(self.lay_max, k)), "stream": torch.cuda.Stream(),
                               "Kst": torch.empty((Hkv, self.G * k, d), dtype=torch.bfloat16, device=dev),
                               "Vst": torch.empty((Hkv, self.G * k, d), dtype=torch.bfloat16, device=dev)})
        self.sess = []
        for n in self.lengths:
            lay = fb.make_layout(Hkv, Hq, n, d)
            rows = dict(pin_memory=True) if host_rows else dict(device=dev)
            self.sess.append({
                "n": n, "lay": lay,
                "hp": torch.empty((Hkv, d, 4, lay.plane_stride_words), dtype=torch.int64, pin_memory=True),
                "hs": torch.empty((Hkv, d, lay.scale_stride), dtype=torch.int16, pin_memory=True),
                "Kr": torch.empty((Hkv, n, d), dtype=torch.bfloat16, **rows), "Vr": torch.empty((Hkv, n, d), dtype=torch.bfloat16, **rows),
                "q": None, "var": None,
                "depth": torch.zeros((Hq // self.hpp, d), dtype=torch.uint8, device=dev),
                "scores": torch.zeros((Hq, lay.score_stride), dtype=torch.float32, device=dev),
                "idx": torch.zeros((Hq, k), dtype=torch.int32, device=dev), "idx_local": torch.zeros((Hq, k), dtype=torch.int32, device=dev),
                "ucount": torch.zeros((Hkv,), dtype=torch.int32, device=dev), "out": torch.zeros((Hq, d), dtype=torch.float32, device=dev)})
        self.planes = torch.empty((Hkv, d, 4, self.lay_max.plane_stride_words), dtype=torch.int64, device=dev)
        self.scales = torch.empty((Hkv, d, self.lay_max.scale_stride), dtype=torch.int16, device=dev)

    def build_layer(self, layer, seed=4, on_session=None):
        """The stores of one layer for every session (not timed: once per sequence).  on_session(i, L, planes, scales) is
        called while the session's generated layer L and its device-side planes are alive."""
        from workloads.synth import make_layer
        Hkv, d = self.Hkv, self.d
        for i, S in enumerate(self.sess):
            L = make_layer(S["n"], Hkv, self.Hq, d, seed=seed, session=i, layer=layer, device=str(self.dev))
            lay = S["lay"]
            pv = self.planes.view(-1)[:Hkv * d * 4 * lay.plane_stride_words].view(Hkv, d, 4, lay.plane_stride_words)
            sv = self.scales.view(-1)[:Hkv * d * lay.scale_stride].view(Hkv, d, lay.scale_stride)
            self.ctx.fathom_build_planes(lay, L.K, pv, sv, self.main)
            S["hp"].copy_(pv); S["hs"].copy_(sv)
            S["Kr"].copy_(L.Krows); S["Vr"].copy_(L.Vrows)
            S["q"], S["var"] = L.q, L.var
            if on_session is not None:
                torch.cuda.synchronize()
                on_session(i, L, pv, sv)
            del L
        torch.cuda.synchronize()

    def decode_layer(self):
        """Enqueues the decode step of the current layer over all sessions; everything is joined back on the main stream."""
        fb, k, hpp, main = self.fb, self.k, self.hpp, self.main
        nl = len(self.lanes)
        sm = 1.0 / math.sqrt(self.d)
        fork = torch.cuda.Event(); fork.record(main)
        for W in self.lanes:
            W["stream"].wait_event(fork)
        for g0 in range(0, len(self.sess), nl):
            grp = self.sess[g0:g0 + nl]
            items = []
            for S in grp:
                self.ctx.fathom_alloc_depth(S["lay"], S["q"], S["var"], fb.DEPTH_WATERFILL, self.B, hpp, S["depth"], main)
                items.append((S["lay"], S["hp"], S["hs"], S["q"], S["depth"], S["scores"]))
            self.ctx.fathom_scan_batch(items, hpp, main)
            done = torch.cuda.Event(); done.record(main)
            for j, S in enumerate(grp):
                W = self.lanes[j]
                st, c = W["stream"], W["ctx"]
                st.wait_event(done)
                c.fathom_topk(S["lay"], S["scores"], k, 0, 0, S["idx"], st)
                c.fathom_gather_union(S["lay"], S["idx"], k, S["Kr"], S["Vr"], W["Kst"], W["Vst"], S["idx_local"], S["ucount"], st)
                c.fathom_sparse_attend(self.lay_stage, S["q"], W["Kst"], W["Vst"], S["idx_local"], k, sm, S["out"], st)
        for W in self.lanes:
            join = torch.cuda.Event(); join.record(W["stream"])
            main.wait_event(join)

    def link_bytes(self):
        """Bytes one decode step of the current layer moves over the host link: plane words and scales of the active
        rows (from the depths the step left behind) and the distinct rows fetched (from the union counts)."""
        pl = 0.0
        for S in self.sess:
            pl += sum(bits_per_token(r) for r in S["depth"].cpu().numpy()) / 8.0 * S["n"] * max(1, self.hpp // 4)
        rows = sum(int(S["ucount"].sum().item()) for S in self.sess) * self.d * 2 * 2
        return pl, float(rows)

    def status(self):
        st = self.ctx.fathom_device_status(self.main)
        for W in self.lanes:
            st |= W["ctx"].fathom_device_status(W["stream"])
        return st

    def close(self):
        self.ctx.close()
        for W in self.lanes:
            W["ctx"].close()


def probe_host_link(dev, stream):
    """One pinned -> device copy of 1 GiB, best of 10: the denominator of every host-link fraction."""
    src = torch.empty(1 << 30, dtype=torch.uint8, pin_memory=True)
    dst = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
    best = 1e9
    for _ in range(10):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream); dst.copy_(src, non_blocking=True); b.record(stream)
        torch.cuda.synchronize()
        best = min(best, a.elapsed_time(b))
    return (1 << 30) / (best * 1e-3) / 1e9


def run_config4(args):
    """Times one decode step per layer over --layers independently seeded layers (default here: all 36) of the 16-session
    batch; reports the per-layer median, the total over the layers measured, and the host-link rate (planes + rows)."""
    from paper_2609_17652_b200 import binding as fb
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    C = Config4(fb, dev, lanes=args.lanes)
    link = probe_host_link(dev, C.main)
    layer_ms, plane_b, row_b = [], [], []
    for layer in range(args.layers):
        C.build_layer(layer)
        ts = []
        for it in range(3):                                      # one untimed pass, then two timed ones of the same layer
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(C.main); C.decode_layer(); b.record(C.main)
            torch.cuda.synchronize()
            if it:
                ts.append(a.elapsed_time(b))
        layer_ms.append(min(ts))
        pb, rb = C.link_bytes()
        plane_b.append(pb); row_b.append(rb)
    # the zero-copy scan alone, session by session (layer: the last one built): link rate against session length
    per_session = []
    for S in C.sess:
        ts = []
        for it in range(4):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(C.main); C.ctx.fathom_scan(S["lay"], S["hp"], S["hs"], S["q"], S["depth"], C.hpp, S["scores"], C.main); b.record(C.main)
            torch.cuda.synchronize()
            if it:
                ts.append(a.elapsed_time(b))
        nbytes = sum(bits_per_token(r) for r in S["depth"].cpu().numpy()) / 8.0 * S["n"]
        g = nbytes / (statistics.median(ts) * 1e-3) / 1e9
        per_session.append({"n": S["n"], "scan_ms": round(statistics.median(ts), 3), "gbs": round(g, 2), "frac_of_measured_link": round(g / link, 3)})
    status = C.status()
    total_tokens = sum(C.lengths)
    med = statistics.median(layer_ms)
    total_b = float(np.mean(plane_b) + np.mean(row_b))
    print(json.dumps({
        "metric": METRIC, "value": total_tokens * C.Hkv / (med * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.layers,
        "ms_per_layer_median": round(med, 3), "ms_per_layer_min": round(min(layer_ms), 3), "ms_per_layer_max": round(max(layer_ms), 3),
        "ms_decode_step_all_layers_measured": round(sum(layer_ms), 2), "layers_measured": args.layers, "higher_is_better": True,
        "dtype": "u64 bit planes + f32 accumulate", "data": "synthetic",
        "config": {"workload": "agentic multi-session batch (config 4): 16 sessions, planes, scales and K/V rows in pinned host memory",
                   "session_tokens": C.lengths, "total_tokens": total_tokens, "kv_heads": C.Hkv, "q_heads": C.Hq, "budget_bits": C.B,
                   "k": C.k, "layers_of_the_model": 36, "stream_lanes": len(C.lanes),
                   "step": "per session: alloc_depth, scan (fathom_scan_batch per group of sessions), topk, gather_union from host rows, "
                           "sparse_attend over the staged rows"},
        "bytes_over_link_per_layer": {"planes_and_scales": float(np.mean(plane_b)), "rows": float(np.mean(row_b)), "total": total_b},
        "host_link_gbs": round(total_b / (med * 1e-3) / 1e9, 2), "link_peak_gbs": round(link, 2),
        "frac_of_measured_link": round(total_b / (med * 1e-3) / 1e9 / link, 4),
        "zero_copy_scan_alone_by_session": per_session, "device_status": status}))
    C.close()


# ------------------------------------------------------------------------------------------------ config 5
def run_config5(args):
    """Budget sweep at n = 1M, 8 KV / 32 Q heads: water-filled depths for B in {32, 40, 48, 64, 80, 136} against the
    fixed-channel mode (top-r channels at all four planes, r = 16 -> 68 bits, r = 32 -> 136 bits) through the same
    kernels.  Per plan: bits per token, bytes read, scan time (L2 flushed), and the relative L2 error of the attention
    output against dense attention over all n rows (the dense reference is a measurement aid computed with plain torch
    ops in fp64 on the stored bf16 rows; it is not part of the library)."""
    from paper_2609_17652_b200 import binding as fb
    from workloads.synth import make_layer
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    n, Hkv, Hq, d, k = args.n, WORKLOAD["Hkv"], WORKLOAD["Hq"], WORKLOAD["d"], args.k
    G = Hq // Hkv
    L = make_layer(n, Hkv, Hq, d, seed=5, device=str(dev))
    lay = fb.make_layout(Hkv, Hq, n, d)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    planes = torch.zeros((Hkv, d, 4, lay.plane_stride_words), dtype=torch.int64, device=dev)
    scales = torch.zeros((Hkv, d, lay.scale_stride), dtype=torch.int16, device=dev)
    ctx.fathom_build_planes(lay, L.K, planes, scales)
    depth = torch.zeros((Hkv, d), dtype=torch.uint8, device=dev)
    scores = torch.zeros((Hq, lay.score_stride), dtype=torch.float32, device=dev)
    idx = torch.zeros((Hq, k), dtype=torch.int32, device=dev)
    out = torch.zeros((Hq, d), dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    st = torch.cuda.current_stream()
    dense = torch.zeros((Hq, d), dtype=torch.float64, device=dev)
    for kv in range(Hkv):                                       # dense attention, one KV head at a time
        Kd, Vd = L.Krows[kv].double(), L.Vrows[kv].double()
        e = (L.q[kv * G:(kv + 1) * G].double() @ Kd.T) / math.sqrt(d)
        dense[kv * G:(kv + 1) * G] = torch.softmax(e, dim=1) @ Vd
        del Kd, Vd, e
    rows = []
    plans = [(fb.DEPTH_WATERFILL, B, f"waterfill B={B}") for B in (32, 40, 48, 64, 80, 136)]
    plans += [(fb.DEPTH_FIXED_TOP_R, r, f"fixed top-{r} channels") for r in (16, 32)]
    for mode, budget, name in plans:
        ctx.fathom_alloc_depth(lay, L.q, L.var, mode, budget, G, depth, st)
        ts = []
        for it in range(8):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(st); ctx.fathom_scan(lay, planes, scales, L.q, depth, G, scores, st); b.record(st)
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(a.elapsed_time(b) * 1e3)
        ctx.fathom_topk(lay, scores, k, 0, 0, idx, st)
        ctx.fathom_sparse_attend(lay, L.q, L.Krows, L.Vrows, idx, k, 1.0 / math.sqrt(d), out, st)
        torch.cuda.synchronize()
        dh = depth.cpu().numpy()
        bits = float(np.mean([bits_per_token(r) for r in dh]))
        err = (torch.linalg.norm(out.double() - dense, dim=1) / torch.linalg.norm(dense, dim=1)).cpu().numpy()
        t_us = statistics.median(ts)
        rows.append({"plan": name, "bits_per_token": round(bits, 2), "bytes_read": bits / 8.0 * n * Hkv,
                     "scan_us_l2_flushed": round(t_us, 1), "gbs_index_bytes_only": round(bits / 8.0 * n * Hkv / (t_us * 1e-6) / 1e9, 1),
                     "attn_rel_l2_err_mean": float(err.mean()), "attn_rel_l2_err_max": float(err.max())})
    status = ctx.fathom_device_status()
    ctx.close()
    print(json.dumps({"metric": METRIC, "unit": UNIT, "n_gpus": 1, "data": "synthetic", "dtype": "u64 bit planes + f32 accumulate",
                      "config": {"workload": "budget sweep (config 5)", "n": n, "kv_heads": Hkv, "q_heads": Hq, "d": d, "k": k,
                                 "heads_per_plan": G},
                      "value": n * Hkv / (rows[2]["scan_us_l2_flushed"] * 1e-6), "value_is": "keys scanned per second by the scan at B = 48",
                      "sweep": rows, "device_status": status,
                      "note": "errors characterise the synthetic recipe (attention mass on planted needles): a head that misses "
                              "a needle is off by about 1; every stage is in parity with the oracle at every budget"}))


# ------------------------------------------------------------------------------------------------ per-layer budgets
PLAN_LEVELS = [24, 32, 40, 48, 64, 80, 96, 128]


def layer_recipe(layer: int):
    """How the synthetic layers of the per-layer budget experiment differ: the spread of the channel scales and the number
    of outlier channels change from layer to layer (a concentrated layer needs fewer bits than a flat one)."""
    his = [4.0, 2.0, 8.0, 1.0, 3.0, 6.0]
    return dict(sigma_lo=0.1, sigma_hi=his[layer % len(his)], n_outliers=[4, 2, 0, 4, 1, 3][layer % 6])


def measure_layer_errors(fb, ctx, lay, layers_inputs, levels, k, hpp, stream):
    """err[l][i]: mean over the query heads of the relative L2 error of the attention output of layer l at budget levels[i]
    (decode step through the library: alloc_depth, scan, topk, sparse_attend) against dense attention over all rows (a
    measurement aid in plain torch fp64 on the stored bf16 rows, not part of the library).  Also returns, per layer and
    level, the bits per token read and the depth sums (the budgets as fathom_alloc_depth granted them)."""
    dev = layers_inputs[0].K.device
    Hkv, Hq, d, n = lay.n_kv_heads, lay.n_q_heads, lay.d, lay.n
    G = Hq // Hkv
    planes = torch.zeros((Hkv, d, 4, lay.plane_stride_words), dtype=torch.int64, device=dev)
    scales = torch.zeros((Hkv, d, lay.scale_stride), dtype=torch.int16, device=dev)
    depth = torch.zeros((Hq // hpp, d), dtype=torch.uint8, device=dev)
    scores = torch.zeros((Hq, lay.score_stride), dtype=torch.float32, device=dev)
    idx = torch.zeros((Hq, k), dtype=torch.int32, device=dev)
    out = torch.zeros((Hq, d), dtype=torch.float32, device=dev)
    err, bits, sums = [], [], []
    for L in layers_inputs:
        ctx.fathom_build_planes(lay, L.K, planes, scales, stream)
        dense = torch.zeros((Hq, d), dtype=torch.float64, device=dev)
        for kv in range(Hkv):
            e = (L.q[kv * G:(kv + 1) * G].double() @ L.Krows[kv].double().T) / math.sqrt(d)
            dense[kv * G:(kv + 1) * G] = torch.softmax(e, dim=1) @ L.Vrows[kv].double()
        row_e, row_b, row_s = [], [], []
        for B in levels:
            ctx.fathom_alloc_depth(lay, L.q, L.var, fb.DEPTH_WATERFILL, B, hpp, depth, stream)
            ctx.fathom_scan(lay, planes, scales, L.q, depth, hpp, scores, stream)
            ctx.fathom_topk(lay, scores, k, 0, 0, idx, stream)
            ctx.fathom_sparse_attend(lay, L.q, L.Krows, L.Vrows, idx, k, 1.0 / math.sqrt(d), out, stream)
            torch.cuda.synchronize()
            rel = torch.linalg.norm(out.double() - dense, dim=1) / torch.linalg.norm(dense, dim=1)
            dh = depth.cpu().numpy()
            row_e.append(float(rel.mean())); row_b.append(float(np.mean([bits_per_token(r) for r in dh])))
            row_s.append([int(r.sum()) for r in dh])
        err.append(row_e); bits.append(row_b); sums.append(row_s)
    return err, bits, sums


def run_plan_layers(args):
    """Per-layer budgets (Sec. 3.4) closed on synthetic data: the error of every layer at every budget level is measured
    through the library, fathom_plan_layer_budgets turns the table into one budget per layer at the target mean, and the
    decode step is run again with those budgets; reported against the flat budget at the same mean."""
    from paper_2609_17652_b200 import binding as fb
    from workloads.synth import make_layer
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    n, Hkv, Hq, d, k, hpp = args.n, WORKLOAD["Hkv"], WORKLOAD["Hq"], WORKLOAD["d"], args.k, WORKLOAD["heads_per_plan"]
    nl, target = args.layers, float(args.budget)
    lay = fb.make_layout(Hkv, Hq, n, d)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    st = torch.cuda.current_stream()
    Ls = [make_layer(n, Hkv, Hq, d, seed=6, layer=l, device=str(dev), **layer_recipe(l)) for l in range(nl)]
    err, bits, sums = measure_layer_errors(fb, ctx, lay, Ls, PLAN_LEVELS, k, hpp, st)
    choice = fb.fathom_plan_layer_budgets(err, PLAN_LEVELS, target)
    planned = [PLAN_LEVELS[c] for c in choice]
    flat_i = PLAN_LEVELS.index(int(target)) if int(target) in PLAN_LEVELS else None
    res = {"metric": "attention_rel_l2_error_at_equal_mean_bits", "unit": "relative L2 error (mean over layers and heads)",
           "data": "synthetic", "n_gpus": 1,
           "config": {"workload": "per-layer budgets (Sec. 3.4) on synthetic layers of varying channel spread", "n": n, "layers": nl,
                      "kv_heads": Hkv, "q_heads": Hq, "k": k, "levels": PLAN_LEVELS, "target_mean_budget": target,
                      "layer_recipes": [layer_recipe(l) for l in range(nl)]},
           "error_table": [[round(e, 5) for e in row] for row in err],
           "planned_budgets": planned, "planned_mean_budget": sum(planned) / nl,
           "planned_mean_error": float(np.mean([err[l][choice[l]] for l in range(nl)])),
           "planned_mean_bits_per_token": float(np.mean([bits[l][choice[l]] for l in range(nl)])),
           "granted_depth_sums_at_planned_budgets": [sums[l][choice[l]] for l in range(nl)]}
    if flat_i is not None:
        res["flat_mean_error"] = float(np.mean([err[l][flat_i] for l in range(nl)]))
        res["flat_mean_bits_per_token"] = float(np.mean([bits[l][flat_i] for l in range(nl)]))
    res["value"] = res["planned_mean_error"]
    res["higher_is_better"] = False
    res["device_status"] = ctx.fathom_device_status()
    ctx.close()
    print(json.dumps(res))


# ------------------------------------------------------------------------------------------------ one stage
STAGES = ["build", "alloc", "scan", "topk", "attend", "scan_topk", "rotate", "rotate_build", "calibrate", "variance", "union", "klt_basis"]


def run_stage(a):
    """Times (or exposes to a profiler) ONE stage of the hot path on synthetic device buffers.  It allocates only what the
    chosen stage touches (random plane words and scales for the scan, random scores for top-k, ...), so a full-size launch
    fits in a few hundred MB and can be captured with ncu.  Values are random but shaped like the real ones; nothing is
    checked here (the tests do that).  Prints one line."""
    from paper_2609_17652_b200 import binding as fb
    dev = torch.device("cuda", 0)
    fb.fathom_scan_set_ctas_per_plan(a.ctas)
    torch.manual_seed(0)
    n, Hkv, Hq, d, hpp = a.n, a.kv_heads, a.q_heads, 128, a.heads_per_plan_arg
    lay = fb.make_layout(Hkv, Hq, n, d)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, a.k))
    q = torch.randn(Hq, d, device=dev)
    var = torch.exp(torch.empty(Hkv, d, device=dev).uniform_(math.log(0.01), math.log(16.0)))
    var[:, :4] = 256.0
    depth = torch.zeros((Hq // hpp, d), dtype=torch.uint8, device=dev)
    ctx.fathom_alloc_depth(lay, q, var, fb.DEPTH_WATERFILL, a.budget, hpp, depth)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    st = torch.cuda.current_stream()

    if a.stage in ("build", "rotate", "rotate_build", "calibrate", "variance"):
        K = torch.randn(Hkv, n, d, device=dev)
    if a.stage in ("rotate", "rotate_build", "calibrate", "variance"):
        mean = torch.zeros(Hkv, d, device=dev)
        cov = torch.zeros(Hkv, d, d, device=dev)
        basis = torch.linalg.qr(torch.randn(Hkv, d, d, device=dev))[0].contiguous()
        K_rot = torch.empty(Hkv, n, d, device=dev) if a.stage == "rotate" else None
    if a.stage == "klt_basis":
        X = torch.randn(Hkv, 4096, d, device=dev) * torch.exp(torch.randn(Hkv, 1, d, device=dev))
        cov = torch.stack([torch.cov((X[h] @ torch.linalg.qr(torch.randn(d, d, device=dev))[0]).T) for h in range(Hkv)]).contiguous()
        basis = torch.empty(Hkv, d, d, device=dev)
        lam = torch.empty(Hkv, d, device=dev)
    if a.stage in ("build", "rotate_build", "scan", "scan_topk"):
        planes = torch.randint(-(1 << 62), 1 << 62, (Hkv, d, 4, lay.plane_stride_words), dtype=torch.int64, device=dev)
        scales = torch.rand(Hkv, d, lay.scale_stride, device=dev).mul_(0.5).add_(0.01).to(torch.float16).view(torch.int16)
        if a.host_planes:
            hp = torch.empty(planes.shape, dtype=planes.dtype, pin_memory=True); hp.copy_(planes)
            hs = torch.empty(scales.shape, dtype=scales.dtype, pin_memory=True); hs.copy_(scales)
            planes, scales = hp, hs
    if a.stage in ("scan", "topk", "scan_topk"):
        scores = torch.randn(Hq, lay.score_stride, device=dev)
        idx = torch.zeros((Hq, a.k), dtype=torch.int32, device=dev)
    if a.stage in ("attend", "union"):
        rows_n = min(n, 1 << 18)                                  # rows are gathered at random: a smaller pool times the same
        lay = fb.make_layout(Hkv, Hq, rows_n, d)
        Kr = torch.randn(Hkv, rows_n, d, device=dev).to(torch.bfloat16)
        Vr = torch.randn(Hkv, rows_n, d, device=dev).to(torch.bfloat16)
        idx = torch.stack([torch.randperm(rows_n, device=dev)[:a.k].sort().values for _ in range(Hq)]).to(torch.int32)
        out = torch.zeros(Hq, d, device=dev)
        if a.stage == "union":
            G = Hq // Hkv
            ctx.close()
            ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, a.k))
            if a.host_rows:
                hK = torch.empty(Kr.shape, dtype=Kr.dtype, pin_memory=True); hK.copy_(Kr)
                hV = torch.empty(Vr.shape, dtype=Vr.dtype, pin_memory=True); hV.copy_(Vr)
                Kr, Vr = hK, hV
            Kst = torch.empty((Hkv, G * a.k, d), dtype=torch.bfloat16, device=dev)
            Vst = torch.empty_like(Kst)
            loc = torch.empty((Hq, a.k), dtype=torch.int32, device=dev)
            cnt = torch.zeros((Hkv,), dtype=torch.int32, device=dev)

    def run():
        if a.stage == "union":
            ctx.fathom_gather_union(lay, idx, a.k, Kr, Vr, Kst, Vst, loc, cnt, st)
        elif a.stage == "klt_basis":
            ctx.fathom_klt_basis(lay, cov, basis, lam, st)
        elif a.stage == "build":
            ctx.fathom_build_planes(lay, K, planes, scales, st)
        elif a.stage == "alloc":
            ctx.fathom_alloc_depth(lay, q, var, fb.DEPTH_WATERFILL, a.budget, hpp, depth, st)
        elif a.stage == "scan":
            ctx.fathom_scan(lay, planes, scales, q, depth, hpp, scores, st)
        elif a.stage == "topk":
            ctx.fathom_topk(lay, scores, a.k, 0, 0, idx, st)
        elif a.stage == "rotate":
            ctx.fathom_rotate_keys(lay, K, mean, basis, K_rot, st)
        elif a.stage == "rotate_build":
            ctx.fathom_build_planes_rotated(lay, K, mean, basis, planes, scales, st)
        elif a.stage == "calibrate":
            ctx.fathom_calibrate(lay, K, mean, cov, st)
        elif a.stage == "variance":
            ctx.fathom_channel_variance(lay, K, mean, cov[:, 0], st)
        elif a.stage == "scan_topk":
            ctx.fathom_scan_topk(lay, planes, scales, q, depth, hpp, a.k, 0, 0, idx, st)
        else:
            ctx.fathom_sparse_attend(lay, q, Kr, Vr, idx, a.k, 1.0 / math.sqrt(d), out, st)

    ts = []
    for it in range(a.iters + 3):
        if not a.no_flush:
            flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for _ in range(a.repeat):
            run()
        e1.record(st)
        torch.cuda.synchronize()
        if it >= 3:
            ts.append(e0.elapsed_time(e1) * 1e3 / a.repeat)
    print(f"stage={a.stage} n={n} budget={a.budget} k={a.k} median_us={statistics.median(ts):.2f} min_us={min(ts):.2f} "
          f"status={ctx.fathom_device_status()}")
    ctx.close()



# ------------------------------------------------------------------------------------------------ oracle legs
def oracle_step(n_s, B, k, hpp, seed, Hkv=None, barrier=None):
    """One decode step of the oracle (alloc_depth, scan, topk, sparse_attend) on a synthetic layer of n_s tokens; the
    store is built first, untimed, as in the GPU arm.  Returns (seconds of the decode step, seconds of the build)."""
    from oracle import fathom_oracle as O
    from workloads.synth import make_layer
    Hkv = WORKLOAD["Hkv"] if Hkv is None else Hkv
    G = WORKLOAD["Hq"] // WORKLOAD["Hkv"]
    L = make_layer(n_s, Hkv, Hkv * G, WORKLOAD["d"], seed=seed, device="cpu")
    K, q, var = L.K.numpy(), L.q.numpy(), L.var.numpy()
    Kr, Vr = L.Krows.float().numpy(), L.Vrows.float().numpy()
    t0 = time.perf_counter()
    planes, scales = O.build_planes(K)
    t_build = time.perf_counter() - t0
    if barrier is not None:
        barrier.wait(timeout=300)
    t0 = time.perf_counter()
    depth = O.alloc_depth(q, var, "waterfill", B, hpp)
    s = O.scan(planes, scales, q, depth, n_s, hpp)
    idx = O.topk(s, k)
    O.sparse_attend(q, Kr, Vr, idx, 1.0 / math.sqrt(WORKLOAD["d"]))
    return time.perf_counter() - t0, t_build


def _oracle_worker(n_s, B, k, hpp, seed, heads, barrier, queue):
    from threadpoolctl import threadpool_limits
    torch.set_num_threads(1)
    with threadpool_limits(limits=1):
        dt, _ = oracle_step(n_s, B, k, hpp, seed, Hkv=heads, barrier=barrier)
    queue.put(dt)


def oracle_all_cores(n_s, B, k, hpp, seed):
    """The same oracle step with the KV heads (independent problems) spread over worker processes, one thread each; the
    oracle itself is unchanged.  Returns (seconds = the slowest worker's decode step after a common barrier, workers)."""
    import multiprocessing as mp
    Hkv = WORKLOAD["Hkv"]
    workers = max(1, min(os.cpu_count() or 1, Hkv))
    while Hkv % workers:
        workers -= 1
    ctx = mp.get_context("spawn")                                # the parent may hold a CUDA context: no fork
    barrier, queue = ctx.Barrier(workers), ctx.Queue()
    procs = [ctx.Process(target=_oracle_worker, args=(n_s, B, k, hpp, seed + 1000 * w, Hkv // workers, barrier, queue))
             for w in range(workers)]
    for p_ in procs:
        p_.start()
    import queue as pyqueue
    dts, deadline = [], time.time() + 600
    try:
        while len(dts) < workers:
            try:
                dts.append(queue.get(timeout=2))
            except pyqueue.Empty:
                if any(p_.exitcode not in (None, 0) for p_ in procs):
                    raise RuntimeError("an oracle worker exited with an error")
                if time.time() > deadline:
                    raise RuntimeError("oracle workers timed out")
    finally:
        for p_ in procs:
            if p_.is_alive() and len(dts) < workers:
                p_.terminate()
            p_.join(timeout=10)
    return max(dts), workers


def cpu_baseline(n_s, B, k, hpp):
    from threadpoolctl import threadpool_limits
    torch.set_num_threads(1)
    with threadpool_limits(limits=1):
        dt, t_build = oracle_step(n_s, B, k, hpp, seed=2)
    keys = n_s * WORKLOAD["Hkv"]
    out = {"value": keys / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": round(dt, 2),
           "config": {"n": n_s, "kv_heads": 8, "q_heads": 32, "d": 128, "budget_bits": B, "k": k, "heads_per_plan": hpp},
           "build_planes_seconds_untimed": round(t_build, 2), "host_cores_available": os.cpu_count(),
           "sample": f"one decode step (alloc_depth, scan, topk, sparse_attend) of the same layer shape at n = {n_s} tokens "
                     f"(8 KV / 32 Q heads, B = {B}, k = {k}), numpy fp64, 1 thread"}
    try:
        dt_all, workers = oracle_all_cores(n_s, B, k, hpp, seed=2)
        out["all_cores"] = {"value": keys / dt_all, "unit": UNIT, "cores": workers, "seconds": round(dt_all, 2),
                            "how": "KV heads spread over worker processes (one thread each), the slowest worker's time after a common barrier"}
    except Exception as e:                                      # report, never hide
        out["all_cores"] = {"error": repr(e)}
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from threadpoolctl import threadpool_limits
    torch.set_num_threads(1)
    n_s, B, hpp = args.ref_sample_tokens, args.budget, WORKLOAD["heads_per_plan"]
    k = min(args.k, 2048)
    with threadpool_limits(limits=1):
        for w in range(args.warmup):
            oracle_step(n_s, B, k, hpp, seed=100 + w)
        ts = [oracle_step(n_s, B, k, hpp, seed=200 + s)[0] for s in range(args.steps)]
    dt = sum(ts) / len(ts)
    val = n_s * WORKLOAD["Hkv"] / dt
    sample = (f"each step = one decode step (alloc_depth, scan, topk, sparse_attend) on one layer of the same shape at n = {n_s} tokens "
              f"(8 KV / 32 Q heads, B = {B}, k = {k}), numpy fp64, 1 thread; a bounded sample of the n = {args.n}, k = {args.k} workload")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(dt * 1e3, 2), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD["name"] + " - bounded sample", "n": n_s, "kv_heads": 8, "q_heads": 32, "d": 128,
                   "budget_bits": B, "k": k, "heads_per_plan": hpp, "sample_of": {"n": args.n, "k": args.k}},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


if __name__ == "__main__":
    a = parse_args()
    if a.layers is None:
        a.layers = 36 if a.config4 else 12
    if a.stage:
        run_stage(a)
    elif a.plan_layers:
        run_plan_layers(a)
    elif a.config4:
        run_config4(a)
    elif a.config5:
        run_config5(a)
    elif a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)

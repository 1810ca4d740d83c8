"""Times (or exposes to a profiler) ONE stage of the hot path on synthetic device buffers.

    python -m paper_2609_17652_b200.probe --stage scan|topk|scan_topk|attend|build|alloc|rotate|rotate_build|calibrate|variance [--n N] [--iters I] [--budget B] [--k K]

Unlike bench.py it allocates only what the chosen stage touches (random plane words and scales for the scan,
random scores for top-k, ...), so a full-size launch fits in a few hundred MB and can be captured with ncu.
Values are random but shaped like the real ones; nothing is checked here (the tests do that).
"""
from __future__ import annotations

import argparse
import math
import statistics

import torch

from . import binding as fb


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--stage", required=True, choices=["build", "alloc", "scan", "topk", "attend", "scan_topk", "rotate", "rotate_build", "calibrate", "variance"])
    ap.add_argument("--n", type=int, default=1 << 20)
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--budget", type=int, default=48)
    ap.add_argument("--k", type=int, default=4096)
    ap.add_argument("--kv-heads", type=int, default=8)
    ap.add_argument("--q-heads", type=int, default=32)
    ap.add_argument("--heads-per-plan", type=int, default=4)
    ap.add_argument("--host-planes", action="store_true", help="planes and scales in pinned host memory")
    ap.add_argument("--ctas", type=int, default=0, help="CTAs per plan of the scan (0 = automatic)")
    ap.add_argument("--no-flush", action="store_true", help="do not write a 256 MB buffer between iterations")
    a = ap.parse_args()
    dev = torch.device("cuda", 0)
    fb.fathom_scan_set_ctas_per_plan(a.ctas)
    torch.manual_seed(0)
    n, Hkv, Hq, d, hpp = a.n, a.kv_heads, a.q_heads, 128, a.heads_per_plan
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
    if a.stage == "attend":
        rows_n = min(n, 1 << 18)                                  # rows are gathered at random: a smaller pool times the same
        lay = fb.make_layout(Hkv, Hq, rows_n, d)
        Kr = torch.randn(Hkv, rows_n, d, device=dev).to(torch.bfloat16)
        Vr = torch.randn(Hkv, rows_n, d, device=dev).to(torch.bfloat16)
        idx = torch.stack([torch.randperm(rows_n, device=dev)[:a.k].sort().values for _ in range(Hq)]).to(torch.int32)
        out = torch.zeros(Hq, d, device=dev)

    def run():
        if a.stage == "build":
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
        e0.record(st); run(); e1.record(st)
        torch.cuda.synchronize()
        if it >= 3:
            ts.append(e0.elapsed_time(e1) * 1e3)
    print(f"stage={a.stage} n={n} budget={a.budget} k={a.k} median_us={statistics.median(ts):.2f} min_us={min(ts):.2f} "
          f"status={ctx.fathom_device_status()}")
    ctx.close()


if __name__ == "__main__":
    main()

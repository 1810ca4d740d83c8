"""Test helper: runs the five C-ABI calls on cuda:0 for one synthetic layer and returns host copies."""
from __future__ import annotations

import math

import numpy as np
import torch


def run_gpu(L, B, k, hpp, mode=0, n_sink=0, n_local=0, ctx=None, rows_dtype=torch.bfloat16, host_planes=False,
            depth_override=None, stages=("build", "alloc", "scan", "topk", "attend"), row_align_bytes=128):
    """L: workloads.synth.LayerInputs with tensors on cuda.  Returns a dict of numpy arrays (tight strides)."""
    from paper_2609_17652_b200 import binding as fb
    dev = L.K.device
    lay = fb.make_layout(L.Hkv, L.Hq, L.n, L.d, row_align_bytes=row_align_bytes)
    nb = (L.n + 63) // 64
    own = ctx is None
    if own:
        ctx = fb.Context(dev.index or 0, fb.fathom_scratch_bytes(lay, k))
    out = {}
    planes = torch.full((L.Hkv, L.d, 4, lay.plane_stride_words), -1, dtype=torch.int64, device=dev)
    scales = torch.full((L.Hkv, L.d, lay.scale_stride), 0x7e00, dtype=torch.int16, device=dev)
    ctx.fathom_build_planes(lay, L.K, planes, scales)
    out["planes"] = planes[..., :nb].cpu().numpy().view(np.uint64)
    out["scales"] = scales[..., :nb].cpu().numpy().view(np.float16)
    out["planes_pad"] = planes[..., nb:].cpu().numpy()
    out["planes_t"], out["scales_t"] = planes, scales            # device tensors, for calls made after this one
    if host_planes:
        hp = torch.empty(planes.shape, dtype=planes.dtype, pin_memory=True); hp.copy_(planes)
        hs = torch.empty(scales.shape, dtype=scales.dtype, pin_memory=True); hs.copy_(scales)
        planes_arg, scales_arg = hp, hs
    else:
        planes_arg, scales_arg = planes, scales
    P = L.Hq // hpp
    depth = torch.full((P, L.d), 255, dtype=torch.uint8, device=dev)
    if depth_override is None:
        ctx.fathom_alloc_depth(lay, L.q, L.var, mode, B, hpp, depth)
    else:
        depth.copy_(torch.as_tensor(depth_override, dtype=torch.uint8))
    out["depth"] = depth.cpu().numpy()
    if "scan" not in stages:
        return out
    scores = torch.full((L.Hq, lay.score_stride), float("nan"), dtype=torch.float32, device=dev)
    ctx.fathom_scan(lay, planes_arg, scales_arg, L.q, depth, hpp, scores)
    out["scores"] = scores[:, :L.n].cpu().numpy()
    out["scores_pad"] = scores[:, L.n:].cpu().numpy()
    if "topk" in stages:
        idx = torch.full((L.Hq, k), -1, dtype=torch.int32, device=dev)
        ctx.fathom_topk(lay, scores, k, n_sink, n_local, idx)
        out["idx"] = idx.cpu().numpy()
        if "attend" in stages:
            o = torch.full((L.Hq, L.d), float("nan"), dtype=torch.float32, device=dev)
            Kr = L.Krows if rows_dtype == torch.bfloat16 else L.K
            Vr = L.Vrows if rows_dtype == torch.bfloat16 else L.Vrows.float()
            ctx.fathom_sparse_attend(lay, L.q, Kr, Vr, idx, k, 1.0 / math.sqrt(L.d), o)
            out["out"] = o.cpu().numpy()
    out["status"] = ctx.fathom_device_status()
    torch.cuda.synchronize()
    if own:
        ctx.close()
    return out


def score_tolerance(ref):
    """|gpu - ref| <= 1e-5 * max(|ref|, rms(ref)) per head (pure relative error is meaningless at zero crossings)."""
    rms = np.sqrt(np.mean(ref.astype(np.float64) ** 2, axis=1, keepdims=True))
    return 1e-5 * np.maximum(np.abs(ref), rms)

"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import fathom_oracle as O
from workloads.synth import make_layer

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from tests._pipeline import run_gpu, score_tolerance


def host(L):
    return {"K": L.K.cpu().numpy(), "q": L.q.cpu().numpy(), "var": L.var.cpu().numpy(),
            "Krows": L.Krows.float().cpu().numpy(), "Vrows": L.Vrows.float().cpu().numpy()}


def check_all(L, B, k, hpp, mode=0, n_sink=0, n_local=0, **kw):
    H = host(L)
    g = run_gpu(L, B, k, hpp, mode=mode, n_sink=n_sink, n_local=n_local, **kw)
    # (1) planes / scales bit-exact; padding untouched
    planes, scales = O.build_planes(H["K"])
    assert np.array_equal(g["scales"].view(np.uint16), scales.view(np.uint16))
    assert np.array_equal(g["planes"], planes)
    assert np.all(g["planes_pad"] == -1)
    # (2) depths bit-exact
    mode_name = {0: "waterfill", 1: "fixed_top_r", 2: "uniform"}[mode]
    depth = O.alloc_depth(H["q"], H["var"], mode_name, B, hpp)
    assert np.array_equal(g["depth"], depth)
    # (3) scores within 1e-5 (relative to max(|s|, rms))
    ref = O.scan(planes, scales, H["q"], depth, L.n, hpp)
    err = np.abs(g["scores"].astype(np.float64) - ref)
    assert np.all(err <= score_tolerance(ref)), float((err / score_tolerance(ref)).max())
    assert np.all(np.isnan(g["scores_pad"]))
    # (4) top-k, stage-isolated: oracle top-k of the GPU's own scores, bit-exact index lists
    idx = O.topk(g["scores"].astype(np.float64), k, n_sink, n_local)
    assert np.array_equal(g["idx"], idx)
    # end to end: sets may differ only inside the tolerance band around the k-th oracle score
    idx_ref = O.topk(ref, k, n_sink, n_local)
    for h in range(L.Hq):
        diff = np.setxor1d(idx_ref[h], g["idx"][h])
        if len(diff):
            kth = np.sort(ref[h])[::-1][k - 1]
            assert np.all(np.abs(ref[h, diff] - kth) <= 4 * score_tolerance(ref)[h].max())
    # (5) attention over the same index lists
    Kr = H["K"] if kw.get("rows_dtype") == torch.float32 else H["Krows"]       # rows at the precision the GPU was given
    o_ref = O.sparse_attend(H["q"], Kr, H["Vrows"], g["idx"], 1.0 / math.sqrt(L.d))
    rel = np.linalg.norm(g["out"] - o_ref, axis=1) / np.linalg.norm(o_ref, axis=1)
    assert rel.max() <= 2e-3, rel.max()
    assert g["status"] == 0
    return g, ref


def test_config1_tiny_single_head():
    L = make_layer(4096, Hkv=1, Hq=1, seed=0, device="cuda")
    g, _ = check_all(L, B=48, k=64, hpp=1)
    assert set(L.needles[0].tolist()) <= set(g["idx"][0].tolist())


@pytest.mark.parametrize("n", [1, 63, 64, 65, 127, 200, 2047, 2049, 4100, 9001])
def test_ragged_lengths(n):
    L = make_layer(n, Hkv=2, Hq=8, seed=n, device="cuda")
    k = max(1, min(n, 37 if n > 40 else n))
    check_all(L, B=48, k=k, hpp=4)


@pytest.mark.parametrize("hpp", [1, 2, 4])
def test_plan_granularity(hpp):
    L = make_layer(5000, Hkv=2, Hq=8, seed=3, device="cuda")
    check_all(L, B=48, k=100, hpp=hpp)


def test_eight_heads_per_plan():
    L = make_layer(3000, Hkv=1, Hq=8, seed=4, device="cuda")
    check_all(L, B=64, k=50, hpp=8)


@pytest.mark.parametrize("mode,budget", [(1, 16), (1, 32), (2, 2), (2, 0), (0, 0), (0, 1), (0, 136), (0, 511), (0, 512), (0, 600)])
def test_depth_modes_and_budgets(mode, budget):
    L = make_layer(4500, Hkv=2, Hq=8, seed=5, device="cuda")
    check_all(L, B=budget, k=77, hpp=4, mode=mode)


def test_sink_and_local_tokens():
    L = make_layer(6000, Hkv=2, Hq=8, seed=6, device="cuda")
    g, _ = check_all(L, B=48, k=128, hpp=4, n_sink=4, n_local=32)
    for h in range(8):
        s = set(g["idx"][h].tolist())
        assert set(range(4)) <= s and set(range(6000 - 32, 6000)) <= s
    check_all(L, B=48, k=36, hpp=4, n_sink=4, n_local=32)       # nothing left to select


def test_all_planes_equals_dense_4bit_dot_product():
    L = make_layer(8192, Hkv=2, Hq=8, seed=7, device="cuda")
    g, _ = check_all(L, B=512, k=256, hpp=4)
    codes, scales = O.quantise_block_codes(L.K.cpu().numpy())
    S = np.repeat(scales.astype(np.float64), 64, axis=2)[:, :, :L.n].transpose(0, 2, 1)
    deq = (codes.astype(np.float64) - 7.5) * S
    qh = L.q.cpu().numpy().astype(np.float64)
    for h in range(8):
        ref = deq[h // 4] @ qh[h]
        assert np.all(np.abs(g["scores"][h] - ref) <= score_tolerance(ref[None])[0])


def test_topk_heavy_ties_and_signed_zero():
    from paper_2609_17652_b200 import binding as fb
    n, Hq = 20000, 4
    lay = fb.make_layout(1, Hq, n)
    r = np.random.default_rng(0)
    s = np.zeros((Hq, lay.score_stride), dtype=np.float32)
    s[0, :n] = np.round(r.standard_normal(n), 1)                # many exact ties
    s[1, :n] = 1.0                                              # all equal: the k lowest indices win
    s[2, :n] = np.where(r.random(n) < 0.5, 0.0, -0.0)           # +0 / -0 are equal
    s[3, :n] = -np.abs(np.round(r.standard_normal(n), 2))       # all non-positive
    sc = torch.from_numpy(s).cuda()
    for k in (1, 5, 1000, 4096):
        ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
        idx = torch.empty((Hq, k), dtype=torch.int32, device="cuda")
        ctx.fathom_topk(lay, sc, k, 0, 0, idx)
        want = O.topk(s[:, :n].astype(np.float64), k)
        assert np.array_equal(idx.cpu().numpy(), want)
        assert ctx.fathom_device_status() == 0
        ctx.close()


def test_attention_fp32_rows_and_k_equals_n():
    L = make_layer(300, Hkv=2, Hq=8, seed=8, device="cuda")
    check_all(L, B=48, k=300, hpp=4, rows_dtype=torch.float32)


def test_planes_in_pinned_host_memory_give_identical_scores():
    L = make_layer(70000, Hkv=2, Hq=8, seed=9, device="cuda")
    a = run_gpu(L, 48, 64, 4, stages=("scan",))
    b = run_gpu(L, 48, 64, 4, stages=("scan",), host_planes=True)
    assert np.array_equal(a["scores"], b["scores"])


@pytest.mark.parametrize("n,Hkv,Hq,B,hpp,ctas", [(70001, 2, 8, 136, 4, 5), (33000, 2, 8, 48, 1, 3), (40000, 1, 8, 200, 8, 1),
                                                 (5000, 2, 8, 80, 2, 2)])
def test_scan_with_few_persistent_ctas_walking_many_tiles(n, Hkv, Hq, B, hpp, ctas):
    """A CTA of the scan walks several tiles and several passes per tile (its next tile's planes fetched ahead into the
    other half of its double buffer): with only `ctas` CTAs per plan the scores are those of the oracle, and bit for
    bit those of the default launch."""
    from paper_2609_17652_b200 import binding as fb
    L = make_layer(n, Hkv=Hkv, Hq=Hq, seed=21, device="cuda")
    a = run_gpu(L, B, 64, hpp, stages=("scan",))
    fb.fathom_scan_set_ctas_per_plan(ctas)
    try:
        b = run_gpu(L, B, 64, hpp, stages=("scan",))
    finally:
        fb.fathom_scan_set_ctas_per_plan(0)
    assert np.array_equal(a["scores"], b["scores"])
    H = host(L)
    planes, scales = O.build_planes(H["K"])
    depth = O.alloc_depth(H["q"], H["var"], "waterfill", B, hpp)
    ref = O.scan(planes, scales, H["q"], depth, n, hpp)
    assert np.all(np.abs(b["scores"].astype(np.float64) - ref) <= score_tolerance(ref))
    assert b["status"] == 0


def test_bf16_keys_build():
    L = make_layer(1000, Hkv=2, Hq=8, seed=10, device="cuda")
    from paper_2609_17652_b200 import binding as fb
    lay = fb.make_layout(2, 8, 1000)
    ctx = fb.Context(0, 0)
    planes = torch.zeros((2, 128, 4, lay.plane_stride_words), dtype=torch.int64, device="cuda")
    scales = torch.zeros((2, 128, lay.scale_stride), dtype=torch.int16, device="cuda")
    ctx.fathom_build_planes(lay, L.Krows, planes, scales)
    torch.cuda.synchronize()
    p_ref, s_ref = O.build_planes(L.Krows.float().cpu().numpy())
    nb = 16
    assert np.array_equal(planes[..., :nb].cpu().numpy().view(np.uint64), p_ref)
    assert np.array_equal(scales[..., :nb].cpu().numpy().view(np.uint16), s_ref.view(np.uint16))
    ctx.close()


def test_argument_validation_returns_codes():
    from paper_2609_17652_b200 import binding as fb
    import ctypes as C
    lay = fb.make_layout(2, 8, 1000)
    ctx = fb.Context(0, 1024)
    x = torch.zeros(4096, dtype=torch.float32, device="cuda")
    with pytest.raises(fb.FathomError) as e:
        ctx.fathom_topk(lay, x, 100, 0, 0, x)
    assert e.value.status == -4                                   # scratch too small
    with pytest.raises(fb.FathomError) as e:
        ctx.fathom_topk(lay, x, 2000, 0, 0, x)
    assert e.value.status == -1                                   # k > n
    bad = fb.make_layout(2, 8, 1000); bad.d = 64
    with pytest.raises(fb.FathomError) as e:
        ctx.fathom_scan(bad, x, x, x, x, 4, x)
    assert e.value.status == -2
    bad = fb.make_layout(2, 8, 1000); bad.plane_stride_words = 17
    with pytest.raises(fb.FathomError) as e:
        ctx.fathom_scan(bad, x, x, x, x, 4, x)
    assert e.value.status == -3
    with pytest.raises(fb.FathomError) as e:
        ctx.fathom_scan(lay, x, x, x, x, 3, x)
    assert e.value.status == -1
    with pytest.raises(fb.FathomError) as e:
        ctx.fathom_scan(lay, 0, x, x, x, 4, x)
    assert e.value.status == -1
    ctx.close()


def test_determinism_two_runs_same_bytes():
    L = make_layer(10000, Hkv=2, Hq=8, seed=11, device="cuda")
    a = run_gpu(L, 48, 256, 4)
    b = run_gpu(L, 48, 256, 4)
    for key in ("planes", "depth", "scores", "idx", "out"):
        assert np.array_equal(a[key], b[key]), key


def test_multi_session_batch_with_host_resident_planes():
    """A small stand-in for the agentic multi-session batch: several sessions of ragged, log-uniform lengths,
    two independently seeded layers each, planes read zero-copy from pinned host memory."""
    from workloads.synth import session_lengths
    lengths = session_lengths(4, lo=1000, hi=20000, seed=3)
    assert len(set(n % 64 for n in lengths)) > 1                       # not forced to multiples of 64
    for s, n in enumerate(lengths):
        for layer in range(2):
            L = make_layer(n, Hkv=2, Hq=8, seed=12, session=s, layer=layer, device="cuda")
            check_all(L, B=48, k=min(256, n), hpp=4, host_planes=True)


def test_non_finite_scores_raise_the_short_flag():
    from paper_2609_17652_b200 import binding as fb
    n, Hq, k = 5000, 2, 64
    lay = fb.make_layout(1, Hq, n)
    s = torch.randn(Hq, lay.score_stride, device="cuda")
    s[1, :n - 10] = float("nan")                                        # head 1 has only 10 finite scores
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    idx = torch.empty((Hq, k), dtype=torch.int32, device="cuda")
    ctx.fathom_topk(lay, s, k, 0, 0, idx)
    assert ctx.fathom_device_status() & fb.DEV_TOPK_SHORT
    got = idx.cpu().numpy()
    assert np.array_equal(got[0], O.topk(s[:1, :n].cpu().numpy().astype(np.float64), k)[0])   # the finite head is unaffected
    assert np.all((got[1] >= 0) & (got[1] < n))                         # padded with a valid index, never out of range
    assert ctx.fathom_device_status() == 0                              # reading the word clears it
    ctx.close()


@pytest.mark.parametrize("rows_on_host,dtype", [(False, torch.bfloat16), (True, torch.bfloat16), (False, torch.float32)])
def test_union_of_winners_fetched_once(rows_on_host, dtype):
    """fathom_gather_union against the oracle (bit-exact lists, counts, positions and staged rows), and attention
    over the staged rows against attention over the original rows (identical)."""
    from paper_2609_17652_b200 import binding as fb
    n, Hkv, Hq, k, G = 9000, 2, 8, 300, 4
    L = make_layer(n, Hkv, Hq, seed=21, device="cuda")
    g = run_gpu(L, 48, k, G)                                            # real top-k lists (heads of a group overlap)
    idx = torch.from_numpy(g["idx"]).cuda()
    Kr = L.Krows if dtype == torch.bfloat16 else L.K
    Vr = L.Vrows if dtype == torch.bfloat16 else L.Vrows.float()
    if rows_on_host:
        hK = torch.empty(Kr.shape, dtype=dtype, pin_memory=True); hK.copy_(Kr)
        hV = torch.empty(Vr.shape, dtype=dtype, pin_memory=True); hV.copy_(Vr)
        Ksrc, Vsrc = hK, hV
    else:
        Ksrc, Vsrc = Kr, Vr
    lay = fb.make_layout(Hkv, Hq, n)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    cap = G * k
    Kst = torch.full((Hkv, cap, 128), 7.0, dtype=dtype, device="cuda")
    Vst = torch.full((Hkv, cap, 128), 7.0, dtype=dtype, device="cuda")
    loc = torch.full((Hq, k), -1, dtype=torch.int32, device="cuda")
    cnt = torch.full((Hkv,), -1, dtype=torch.int32, device="cuda")
    ctx.fathom_gather_union(lay, idx, k, Ksrc, Vsrc, Kst, Vst, loc, cnt, row_dtype=fb.BF16 if dtype == torch.bfloat16 else fb.F32)
    # attention over the staged rows (layout with n = G * k) vs attention over the original rows
    lay2 = fb.make_layout(Hkv, Hq, cap)
    o_direct = torch.zeros((Hq, 128), device="cuda"); o_staged = torch.zeros((Hq, 128), device="cuda")
    ctx.fathom_sparse_attend(lay, L.q, Kr, Vr, idx, k, 1 / math.sqrt(128), o_direct)
    torch.cuda.synchronize()
    ctx.fathom_sparse_attend(lay2, L.q, Kst, Vst, loc, k, 1 / math.sqrt(128), o_staged)
    torch.cuda.synchronize()
    assert ctx.fathom_device_status() == 0
    ctx.close()
    ul, Ks, Vs, loc_ref = O.gather_union(g["idx"], G, Kr.float().cpu().numpy(), Vr.float().cpu().numpy())
    assert np.array_equal(cnt.cpu().numpy(), [len(u) for u in ul])
    assert np.array_equal(loc.cpu().numpy(), loc_ref)
    for kv in range(Hkv):
        c = len(ul[kv])
        assert c < cap                                                  # the group's picks do overlap
        assert np.array_equal(Kst[kv, :c].float().cpu().numpy(), Ks[kv])
        assert np.array_equal(Vst[kv, :c].float().cpu().numpy(), Vs[kv])
        assert np.all(Kst[kv, c:].float().cpu().numpy() == 7.0)         # rows past the union are untouched
    assert np.array_equal(o_direct.cpu().numpy(), o_staged.cpu().numpy())


def test_appending_keys_rebuilds_only_the_tail():
    """Incremental append (the paper is silent; a serving stack needs it): new keys can raise the maximum of the
    last, partly filled block, so that block is re-quantised.  Rebuilding from a block index that is a multiple of
    8 keeps every pointer 16-byte aligned, and the result equals a build of the whole sequence."""
    from paper_2609_17652_b200 import binding as fb
    Hkv, n1, n2 = 2, 5000, 5300                                        # 5000 tokens, then 300 more
    L = make_layer(n2, Hkv, 8, seed=31, device="cuda")
    lay2 = fb.make_layout(Hkv, 8, n2)
    ctx = fb.Context(0, 0)
    shape_p, shape_s = (Hkv, 128, 4, lay2.plane_stride_words), (Hkv, 128, lay2.scale_stride)
    full_p = torch.zeros(shape_p, dtype=torch.int64, device="cuda"); full_s = torch.zeros(shape_s, dtype=torch.int16, device="cuda")
    ctx.fathom_build_planes(lay2, L.K, full_p, full_s)
    # store built for the first n1 tokens (same strides, sized for n2) ...
    inc_p = torch.zeros(shape_p, dtype=torch.int64, device="cuda"); inc_s = torch.zeros(shape_s, dtype=torch.int16, device="cuda")
    lay1 = fb.make_layout(Hkv, 8, n1)
    lay1.plane_stride_words, lay1.scale_stride = lay2.plane_stride_words, lay2.scale_stride
    K1 = L.K[:, :n1].contiguous()
    ctx.fathom_build_planes(lay1, K1, inc_p, inc_s)
    # ... then the tail from block b0 = 8 * floor(floor(n1 / 64) / 8) on, one KV head at a time (a head's tokens are
    # contiguous in K, and its plane / scale rows keep their strides)
    b0 = (n1 // 64) // 8 * 8
    tail = fb.make_layout(1, 1, n2 - b0 * 64)
    tail.plane_stride_words, tail.scale_stride = lay2.plane_stride_words, lay2.scale_stride
    for kv in range(Hkv):
        ctx.fathom_build_planes(tail, L.K[kv, b0 * 64:].contiguous(), inc_p[kv, :, :, b0:].data_ptr(), inc_s[kv, :, b0:].data_ptr(),
                                k_dtype=fb.F32)
    torch.cuda.synchronize()
    nb = (n2 + 63) // 64
    assert torch.equal(inc_p[..., :nb], full_p[..., :nb]) and torch.equal(inc_s[..., :nb], full_s[..., :nb])
    ctx.close()


def _fused_vs_unfused(L, B, k, hpp, mode=0, n_sink=0, n_local=0):
    from paper_2609_17652_b200 import binding as fb
    lay = fb.make_layout(L.Hkv, L.Hq, L.n)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    dev = L.K.device
    planes = torch.zeros((L.Hkv, 128, 4, lay.plane_stride_words), dtype=torch.int64, device=dev)
    scales = torch.zeros((L.Hkv, 128, lay.scale_stride), dtype=torch.int16, device=dev)
    ctx.fathom_build_planes(lay, L.K, planes, scales)
    depth = torch.zeros((L.Hq // hpp, 128), dtype=torch.uint8, device=dev)
    ctx.fathom_alloc_depth(lay, L.q, L.var, mode, B, hpp, depth)
    scores = torch.zeros((L.Hq, lay.score_stride), dtype=torch.float32, device=dev)
    want = torch.full((L.Hq, k), -1, dtype=torch.int32, device=dev)
    got = torch.full((L.Hq, k), -2, dtype=torch.int32, device=dev)
    ctx.fathom_scan(lay, planes, scales, L.q, depth, hpp, scores)
    ctx.fathom_topk(lay, scores, k, n_sink, n_local, want)
    torch.cuda.synchronize()
    ctx.fathom_scan_topk(lay, planes, scales, L.q, depth, hpp, k, n_sink, n_local, got)
    torch.cuda.synchronize()
    assert ctx.fathom_device_status() == 0
    ctx.close()
    assert torch.equal(got, want)
    return scores[:, :L.n].cpu().numpy(), got.cpu().numpy()


@pytest.mark.parametrize("n,k,hpp", [(40000, 300, 4), (40000, 300, 1), (70001, 1000, 2), (9000, 64, 4), (20000, 4096, 4), (300, 300, 4)])
def test_fused_scan_topk_equals_scan_then_topk(n, k, hpp):
    """The fused entry point (threshold from a sampled scan, filtering scan, candidate select) must return exactly
    the lists of fathom_scan + fathom_topk, which are themselves checked against the oracle; sampled path (n >= 16
    tiles and >= 2 k sampled tokens) and dense fallback (short sequences) are both covered."""
    L = make_layer(n, Hkv=2, Hq=8, seed=n + k, device="cuda")
    s, idx = _fused_vs_unfused(L, 48, k, hpp)
    assert np.array_equal(idx, O.topk(s.astype(np.float64), k))


def test_fused_scan_topk_random_shapes():
    """Thirty seeded draws of (n, KV heads, group size, heads per plan, budget, k, forced tokens): fathom_topk of the
    scan's scores and fathom_scan_topk must both give the oracle's selection of those scores."""
    from paper_2609_17652_b200 import binding as fb
    r = np.random.default_rng(3)
    for it in range(30):
        n = int(r.choice([300, 5000, 20000, 40001, 70001, 131072, 200003, 400000, 1048576]))
        Hkv, G = [(1, 4), (2, 4), (1, 8), (2, 2), (1, 1), (4, 4)][int(r.integers(0, 6))]
        Hq = Hkv * G
        hpp = int(r.choice([h for h in (1, 2, 4, 8) if G % h == 0]))
        B = int(r.choice([16, 48, 80, 136, 200]))
        k = max(1, min(int(r.choice([64, 300, 1000, 2048, 4096, 8192])), n // 2))
        n_sink, n_local = (0, 0) if r.random() < 0.5 else (int(r.integers(0, 5)), int(r.integers(0, 40)))
        if n_sink + n_local > k:
            n_sink, n_local = 0, 0
        L = make_layer(n, Hkv, Hq, seed=100 + it, device="cuda")
        g = run_gpu(L, B, k, hpp, n_sink=n_sink, n_local=n_local, stages=("scan", "topk"))
        ref = O.topk(g["scores"].astype(np.float64), k, n_sink, n_local)
        case = (it, n, Hkv, Hq, hpp, B, k, n_sink, n_local)
        assert np.array_equal(g["idx"], ref), case
        lay = fb.make_layout(Hkv, Hq, n)
        ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
        idx = torch.full((Hq, k), -1, dtype=torch.int32, device="cuda")
        ctx.fathom_scan_topk(lay, g["planes_t"], g["scales_t"], L.q, torch.from_numpy(g["depth"]).cuda(), hpp, k, n_sink, n_local, idx)
        assert np.array_equal(idx.cpu().numpy(), ref), case
        assert ctx.fathom_device_status() == 0, case
        ctx.close()


def test_fused_scan_topk_with_forced_tokens_and_degenerate_scores():
    L = make_layer(50000, Hkv=2, Hq=8, seed=77, device="cuda")
    _fused_vs_unfused(L, 48, 200, 4, n_sink=4, n_local=32)
    _fused_vs_unfused(L, 16, 500, 4, mode=1)                           # fixed-channel plan
    _fused_vs_unfused(L, 0, 100, 4)                                    # B = 0: all scores equal, every token is a candidate
    # scores that grow along the sequence: the sampled tiles see the trend, the bound stays a bound
    L.K[:, :, :] = L.K * torch.linspace(0.2, 3.0, L.n, device="cuda")[None, :, None]
    _fused_vs_unfused(L, 48, 400, 4)
    # keys five times larger in the sampled tiles (every 16th tile of 1024 tokens) than elsewhere: the estimate from the
    # sample is far too high, the first filtering scan collects too few, and the second one (bound threshold) must serve
    L2 = make_layer(70000, Hkv=2, Hq=8, seed=78, device="cuda")
    tile = torch.arange(L2.n, device="cuda") // 1024
    L2.K[:, :, :] = L2.K * torch.where(tile % 16 == 0, 5.0, 1.0)[None, :, None]
    _fused_vs_unfused(L2, 48, 600, 4)
    _fused_vs_unfused(L2, 48, 600, 1)


@pytest.mark.parametrize("n", [5000, 8192 + 77])
def test_klt_rotated_store(n):
    """Session calibration, rotation of keys and queries against the oracle, and the rotated variant end to end:
    planes of (K - mu) V, importance from q V and the eigenvalues, same scan / top-k / attention."""
    from paper_2609_17652_b200 import binding as fb
    Hkv, Hq, G, k = 2, 8, 4, 128
    L = make_layer(n, Hkv, Hq, seed=41, device="cuda")
    mix = torch.linalg.qr(torch.randn(Hkv, 128, 128, device="cuda"))[0]          # correlate the channels
    K = (torch.bmm(L.K, mix) + 0.5).contiguous()
    lay = fb.make_layout(Hkv, Hq, n)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    mean = torch.zeros((Hkv, 128), device="cuda"); cov = torch.zeros((Hkv, 128, 128), device="cuda")
    ctx.fathom_calibrate(lay, K, mean, cov)
    torch.cuda.synchronize()
    Kh = K.cpu().numpy()
    mu_ref, C_ref = O.calibrate(Kh)
    assert np.allclose(mean.cpu().numpy(), mu_ref, rtol=1e-5, atol=1e-5)
    scale = np.abs(C_ref).max(axis=(1, 2), keepdims=True)
    assert np.all(np.abs(cov.cpu().numpy() - C_ref) <= 2e-5 * scale)
    # basis from the oracle's eigen-decomposition of the GPU's own statistics (stage isolation)
    V_ref, lam_ref = O.klt_basis(cov.cpu().numpy().astype(np.float64))
    V = torch.from_numpy(V_ref.astype(np.float32)).cuda().contiguous()
    lam = torch.from_numpy(lam_ref.astype(np.float32)).cuda().contiguous()
    K_rot = torch.full((Hkv, n, 128), float("nan"), device="cuda"); q_rot = torch.zeros((Hq, 128), device="cuda")
    ctx.fathom_rotate_keys(lay, K, mean, V, K_rot)
    ctx.fathom_rotate_query(lay, L.q, V, q_rot)
    torch.cuda.synchronize()
    Kr_ref = O.rotate_keys(Kh, mean.cpu().numpy(), V.cpu().numpy())
    rown = np.linalg.norm(Kr_ref, axis=2, keepdims=True)
    assert np.all(np.abs(K_rot.cpu().numpy() - Kr_ref) <= 1e-5 * rown + 1e-6)
    qr_ref = O.rotate_query(L.q.cpu().numpy(), V.cpu().numpy(), G)
    assert np.allclose(q_rot.cpu().numpy(), qr_ref, rtol=1e-5, atol=1e-5)
    ctx.close()
    # the rest of the path on the rotated store, checked stage by stage against the oracle
    L.K, L.q, L.var = K_rot, q_rot, lam
    g, ref = check_all(L, B=48, k=k, hpp=G)
    assert np.all(g["depth"].sum(1) == 48)


@pytest.mark.parametrize("case", ["keys", "few_keys", "identity", "blocks"])
def test_klt_basis_on_the_device(case):
    """fathom_klt_basis against the oracle's eigen-decomposition on what does not depend on signs or on the order inside
    (nearly) equal eigenvalues: the eigenvalues themselves, V^T V = I, V diag(lambda) V^T = C, the directions of
    well-separated eigenvalues; covariances of correlated keys, of fewer keys than channels (rank-deficient), the
    identity (fully degenerate) and a block matrix with repeated eigenvalues."""
    from paper_2609_17652_b200 import binding as fb
    Hkv, Hq = 2, 8
    g = torch.Generator(device="cuda").manual_seed(5)
    if case in ("keys", "few_keys"):
        n = 5000 if case == "keys" else 60
        L = make_layer(max(n, 256), Hkv, Hq, seed=43, device="cuda")
        mix = torch.linalg.qr(torch.randn(Hkv, 128, 128, generator=g, device="cuda"))[0]
        K = (torch.bmm(L.K[:, :n], mix) + 0.25).contiguous()
        C = torch.stack([torch.cov(K[h].double().T) for h in range(Hkv)]).float().contiguous()
    elif case == "identity":
        C = torch.eye(128, device="cuda").repeat(Hkv, 1, 1).contiguous()
    else:
        B4 = torch.tensor([[2.0, 1.0, 0, 0], [1.0, 2.0, 0, 0], [0, 0, 5.0, 0], [0, 0, 0, 5.0]], device="cuda")
        C = torch.block_diag(*[B4] * 32).repeat(Hkv, 1, 1).contiguous()
    lay = fb.make_layout(Hkv, Hq, 1000)
    ctx = fb.Context(0, 0)
    V = torch.full((Hkv, 128, 128), float("nan"), device="cuda"); lam = torch.full((Hkv, 128), float("nan"), device="cuda")
    ctx.fathom_klt_basis(lay, C, V, lam)
    V2 = torch.empty_like(V); lam2 = torch.empty_like(lam)
    ctx.fathom_klt_basis(lay, C, V2, lam2)
    torch.cuda.synchronize()
    assert torch.equal(V, V2) and torch.equal(lam, lam2)                       # bit-reproducible
    assert ctx.fathom_device_status() == 0
    ctx.close()
    Ch = C.cpu().numpy().astype(np.float64)
    Ch = 0.5 * (Ch + Ch.transpose(0, 2, 1))
    V_ref, lam_ref = O.klt_basis(Ch)
    Vh, lh = V.cpu().numpy().astype(np.float64), lam.cpu().numpy().astype(np.float64)
    for h in range(Hkv):
        top = max(lam_ref[h].max(), 1e-30)
        assert np.all(np.diff(lh[h]) <= 0) and np.all(lh[h] >= 0)
        assert np.all(np.abs(lh[h] - lam_ref[h]) <= 1e-5 * top)
        assert np.abs(Vh[h].T @ Vh[h] - np.eye(128)).max() <= 2e-5
        assert np.abs(Vh[h] @ np.diag(lh[h]) @ Vh[h].T - Ch[h]).max() <= 2e-5 * np.abs(Ch[h]).max()
        assert np.all(Vh[h][np.abs(Vh[h]).argmax(axis=0), np.arange(128)] > 0)  # every direction's largest component is positive
        gap = np.minimum(np.abs(np.diff(lam_ref[h], prepend=np.inf)), np.abs(np.diff(lam_ref[h], append=-np.inf)))
        for j in np.nonzero(gap > 1e-3 * top)[0]:                             # a well-separated eigenvalue fixes its direction
            assert abs(Vh[h][:, j] @ V_ref[h][:, j]) >= 1 - 1e-4, (h, j)


def test_rotated_store_built_with_library_calls_only():
    """Session calibration end to end on the device: fathom_calibrate -> fathom_klt_basis -> fathom_rotate_keys /
    fathom_rotate_query, then the five calls on the rotated store, every stage against the oracle on the stage's own input."""
    from paper_2609_17652_b200 import binding as fb
    n, Hkv, Hq, G, k = 9000, 2, 8, 4, 128
    L = make_layer(n, Hkv, Hq, seed=47, device="cuda")
    mix = torch.linalg.qr(torch.randn(Hkv, 128, 128, device="cuda"))[0]
    K = (torch.bmm(L.K, mix) + 0.5).contiguous()
    lay = fb.make_layout(Hkv, Hq, n)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    mean = torch.zeros((Hkv, 128), device="cuda"); cov = torch.zeros((Hkv, 128, 128), device="cuda")
    V = torch.zeros((Hkv, 128, 128), device="cuda"); lam = torch.zeros((Hkv, 128), device="cuda")
    K_rot = torch.full((Hkv, n, 128), float("nan"), device="cuda"); q_rot = torch.zeros((Hq, 128), device="cuda")
    ctx.fathom_calibrate(lay, K, mean, cov)
    ctx.fathom_klt_basis(lay, cov, V, lam)
    ctx.fathom_rotate_keys(lay, K, mean, V, K_rot)
    ctx.fathom_rotate_query(lay, L.q, V, q_rot)
    torch.cuda.synchronize()
    assert ctx.fathom_device_status() == 0
    ctx.close()
    Kh = K.cpu().numpy()
    Kr_ref = O.rotate_keys(Kh, mean.cpu().numpy(), V.cpu().numpy())
    rown = np.linalg.norm(Kr_ref, axis=2, keepdims=True)
    assert np.all(np.abs(K_rot.cpu().numpy() - Kr_ref) <= 1e-5 * rown + 1e-6)
    # the rotated keys are decorrelated: their covariance is diag(lambda) up to the accuracy of the statistics
    Cr = np.stack([np.cov(Kr_ref[h].T) for h in range(Hkv)])
    lh = lam.cpu().numpy().astype(np.float64)
    for h in range(Hkv):
        assert np.abs(Cr[h] - np.diag(lh[h])).max() <= 1e-4 * lh[h].max()
    # scores are preserved up to the constant q . mu (Sec. 3.5): q'.k' + q.mu = q.k
    qh, muh = L.q.cpu().numpy().astype(np.float64), mean.cpu().numpy().astype(np.float64)
    i = np.arange(0, n, 997)
    for hq in range(Hq):
        kv = hq // G
        lhs = Kr_ref[kv][i] @ q_rot.cpu().numpy().astype(np.float64)[hq] + qh[hq] @ muh[kv]
        rhs = Kh[kv][i].astype(np.float64) @ qh[hq]
        assert np.all(np.abs(lhs - rhs) <= 1e-4 * np.linalg.norm(Kh[kv][i], axis=1) * np.linalg.norm(qh[hq]))
    L.K, L.q, L.var = K_rot, q_rot, lam
    g_, ref = check_all(L, B=48, k=k, hpp=G)
    assert np.all(g_["depth"].sum(1) == 48)


@pytest.mark.parametrize("n,dtype", [(1, torch.float32), (777, torch.float32), (1024, torch.float32), (40000 + 13, torch.float32),
                                     (9000, torch.bfloat16)])
def test_channel_variance_kernel(n, dtype):
    """Per-channel mean and unbiased variance of the session's keys against the oracle's written-out definition,
    with a large common offset (the case a one-pass sum of squares gets wrong), several tiles and a ragged tail;
    then the depths planned from the kernel's variances equal those from the oracle's."""
    from paper_2609_17652_b200 import binding as fb
    Hkv, Hq = 2, 8
    L = make_layer(max(n, 64), Hkv, Hq, seed=77, device="cuda")
    K = (L.K[:, :n] + 40.0).to(dtype).contiguous()
    lay = fb.make_layout(Hkv, Hq, n)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, 1))
    mean = torch.full((Hkv, 128), float("nan"), device="cuda"); var = torch.full((Hkv, 128), float("nan"), device="cuda")
    ctx.fathom_channel_variance(lay, K, mean, var)
    ctx.fathom_channel_variance(lay, K, mean, var)                             # scratch reuse
    torch.cuda.synchronize()
    mu_ref, var_ref = O.channel_variance(K.float().cpu().numpy())
    sd = np.sqrt(var_ref)
    assert np.all(np.abs(mean.cpu().numpy() - mu_ref) <= 1e-6 * np.abs(mu_ref) + 1e-5 * sd)
    assert np.all(np.abs(var.cpu().numpy() - var_ref) <= 1e-5 * var_ref)
    if n > 1:
        # the chain fathom_channel_variance -> fathom_alloc_depth on the device, bit-exact against the oracle's depths from
        # the oracle's variances except where the 1e-5 of the variance can change the ranking: channels whose priority
        # g_j 4^-m lies within 2e-5 (relative) of the cut.  Those are counted and reported, never waved through in bulk.
        depth = torch.full((Hq // 4, 128), 255, dtype=torch.uint8, device="cuda")
        ctx.fathom_alloc_depth(lay, L.q, var, fb.DEPTH_WATERFILL, 48, 4, depth)
        torch.cuda.synchronize()
        d_gpu = depth.cpu().numpy()
        q_h = L.q.cpu().numpy()
        assert np.array_equal(d_gpu, O.alloc_depth(q_h, var.cpu().numpy(), "waterfill", 48, 4))   # the kernel on its own input
        d_ref = O.alloc_depth(q_h, var_ref.astype(np.float32), "waterfill", 48, 4)
        g = O.importance(q_h, var_ref.astype(np.float32), 4)
        near = 0
        for p_ in range(d_ref.shape[0]):
            pri = np.sort((g[p_][:, None] * 4.0 ** -np.arange(1, 5)[None, :]).ravel())[::-1]
            cut = 0.5 * (pri[47] + pri[48])
            for j in np.nonzero(d_gpu[p_] != d_ref[p_])[0]:
                m = max(d_gpu[p_][j], d_ref[p_][j])                            # the plane granted on one side only
                assert abs(g[p_][j] * 4.0 ** -float(m) - cut) <= 2e-5 * cut + abs(pri[47] - pri[48]), (p_, j)
                near += 1
        assert np.all(d_gpu.sum(1) == 48)
        assert near <= 4, near
    ctx.close()


@pytest.mark.parametrize("n,B", [(70001, 48), (5000, 80), (3001, 200)])
def test_tight_strides_give_what_line_aligned_strides_give(n, B):
    """The layout only asks for 16-byte strides; rows that start in the middle of a memory line (and stages whose copies
    straddle lines) must give the same planes, scores, picks and outputs as the 128-byte-aligned default."""
    L = make_layer(n, Hkv=2, Hq=8, seed=13, device="cuda")
    a = run_gpu(L, B, 64, 4)
    b = run_gpu(L, B, 64, 4, row_align_bytes=16)
    for key in ("planes", "scales", "depth", "scores", "idx", "out"):
        assert np.array_equal(a[key], b[key]), key
    assert a["status"] == 0 and b["status"] == 0


def test_depths_above_four_are_read_as_four():
    """A depth buffer that was never written (255s) must not send the scan past its row list: it scans like all-4."""
    from paper_2609_17652_b200 import binding as fb
    L = make_layer(3000, Hkv=2, Hq=8, seed=31, device="cuda")
    a = run_gpu(L, 48, 64, 4, stages=("scan",), depth_override=np.full((2, 128), 4, dtype=np.uint8))
    b = run_gpu(L, 48, 64, 4, stages=("scan",), depth_override=np.full((2, 128), 255, dtype=np.uint8))
    assert np.array_equal(a["scores"], b["scores"]) and b["status"] == 0


def test_a_wait_that_runs_out_sets_the_status_bit_and_leaves_the_context_usable():
    """The give-up path of the bounded device-side waits: a barrier that nothing completes (no asynchronous operation
    outstanding) is polled 200 times, the kernel reports FATHOM_DEV_WAIT_EXPIRED and returns; the next calls work."""
    from paper_2609_17652_b200 import binding as fb
    L = make_layer(2000, Hkv=1, Hq=4, seed=3, device="cuda")
    lay = fb.make_layout(1, 4, 2000)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, 64))
    assert ctx.fathom_device_status() == 0
    ctx.fathom_selftest_wait_expiry(200)
    assert ctx.fathom_device_status() == fb.DEV_WAIT_EXPIRED
    assert ctx.fathom_device_status() == 0                                     # reading clears it
    g = run_gpu(L, 48, 64, 4, ctx=ctx, stages=("scan",))
    assert g["status"] == 0 and np.all(np.isfinite(g["scores"]))
    ctx.close()


@pytest.mark.parametrize("n_sink,n_local", [(0, 0), (4, 32)])
def test_topk_single_pass_and_its_exact_fallback(n_sink, n_local):
    """Long rows take the single-pass path (threshold estimated from every 16th 1024-score chunk, candidates
    collected in one read, exact selection among them).  Rows built so that the estimate is right, far too high
    (only the sampled chunks hold high scores: too few candidates -> the exact two-pass path must take over on
    the device), far too low (sampled chunks hold the lowest scores: nearly every token is a candidate) and
    degenerate (all equal, heavy ties) must all give the oracle's selection."""
    from paper_2609_17652_b200 import binding as fb
    n, Hq, k = 200_000 + 37, 6, 3000
    lay = fb.make_layout(1, Hq, n)
    r = np.random.default_rng(21)
    s = np.zeros((Hq, lay.score_stride), dtype=np.float32)
    pos = np.arange(n)
    sampled = (pos // 1024) % 16 == 0
    s[0, :n] = r.standard_normal(n)                                              # estimate about right
    s[1, :n] = np.where(sampled, 10.0, -10.0) + r.standard_normal(n)             # estimate far too high
    s[2, :n] = np.where(sampled, -10.0, 10.0) + r.standard_normal(n)             # estimate far too low
    s[3, :n] = 2.5                                                                # all equal
    s[4, :n] = np.round(r.standard_normal(n), 1)                                  # heavy ties
    s[5, :n] = r.standard_normal(n) * np.where(pos < n // 2, 0.1, 3.0)            # spread changes along the row
    sc = torch.from_numpy(s).cuda()
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    idx = torch.empty((Hq, k), dtype=torch.int32, device="cuda")
    want = O.topk(s[:, :n].astype(np.float64), k, n_sink, n_local)
    for rows in ([0, 3, 4, 5], [0, 1, 2, 3, 4, 5]):          # without and with a head that forces the fall-back
        sub = sc[rows].contiguous()
        lay_sub = fb.make_layout(1, len(rows), n)
        out = torch.full((len(rows), k), -1, dtype=torch.int32, device="cuda")
        for _ in range(2):                                   # scratch reuse
            ctx.fathom_topk(lay_sub, sub, k, n_sink, n_local, out)
        assert np.array_equal(out.cpu().numpy(), want[rows])
        assert ctx.fathom_device_status() == 0
    ctx.close()


@pytest.mark.parametrize("n,dtype", [(1, torch.float32), (100, torch.float32), (128, torch.float32), (64 * 75 + 1, torch.bfloat16),
                                     (20000, torch.float32)])
@pytest.mark.parametrize("path", ["tensor", "simt"])
def test_rotation_and_covariance_kernels_both_paths(n, dtype, path, monkeypatch):
    """fathom_calibrate and fathom_rotate_keys on the tensor cores (split tf32 operands) and as plain fp32 kernels,
    each against the oracle, over tiny, ragged and multi-tile sequences, fp32 and bf16 keys, three KV heads (the
    tile ranges of the persistent CTAs then straddle heads)."""
    from paper_2609_17652_b200 import binding as fb
    if path == "simt":
        monkeypatch.setenv("FATHOM_ROTATE_PATH", "simt"); monkeypatch.setenv("FATHOM_CALIBRATE_PATH", "simt")
    Hkv, Hq = 3, 6
    g = torch.Generator(device="cuda"); g.manual_seed(1000 + n)
    mix = torch.linalg.qr(torch.randn(Hkv, 128, 128, device="cuda", generator=g))[0]
    sig = torch.exp(torch.rand(Hkv, 1, 128, device="cuda", generator=g) * 3.0 - 2.0)
    K = (torch.bmm(torch.randn(Hkv, n, 128, device="cuda", generator=g) * sig, mix) + 1.5).to(dtype).contiguous()
    lay = fb.make_layout(Hkv, Hq, n)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, 1))
    mean = torch.full((Hkv, 128), float("nan"), device="cuda"); cov = torch.full((Hkv, 128, 128), float("nan"), device="cuda")
    ctx.fathom_calibrate(lay, K, mean, cov)
    Kh = K.float().cpu().numpy()
    mu_ref, C_ref = O.calibrate(Kh)
    assert np.allclose(mean.cpu().numpy(), mu_ref, rtol=1e-5, atol=1e-5)
    scale = np.maximum(np.abs(C_ref).max(axis=(1, 2), keepdims=True), 1e-30)
    assert np.all(np.abs(cov.cpu().numpy() - C_ref) <= 2e-5 * scale)
    V = torch.linalg.qr(torch.randn(Hkv, 128, 128, device="cuda", generator=g))[0].contiguous()
    K_rot = torch.full((Hkv, n, 128), float("nan"), device="cuda")
    ctx.fathom_rotate_keys(lay, K, mean, V, K_rot)
    ctx.fathom_rotate_keys(lay, K, mean, V, K_rot)                               # scratch reuse
    torch.cuda.synchronize()
    Kr_ref = O.rotate_keys(Kh, mean.cpu().numpy(), V.cpu().numpy())
    rown = np.linalg.norm(Kr_ref, axis=2, keepdims=True)
    assert np.all(np.abs(K_rot.cpu().numpy() - Kr_ref) <= 1e-5 * rown + 1e-6)
    assert ctx.fathom_device_status() == 0
    ctx.close()


@pytest.mark.parametrize("n,Hq,k,n_sink,n_local", [(300_000, 3, 6000, 0, 0),      # lists of 8192..16384: two rounds of loads
                                                   (300_000, 3, 2500, 4, 32),   # short lists, forced tokens
                                                   (1_700_000, 2, 2048, 0, 0),  # four bitmap groups per thread
                                                   (2_097_151, 1, 4096, 0, 0),  # the longest sequence of the short way (tokens in 21 bits)
                                                   (2_097_152 + 64, 1, 4096, 3, 40),   # one more block: the general way
                                                   (140_000, 2, 1024, 0, 64)])  # a sample of few chunks
def test_topk_direct_select_short_and_general_way(n, Hq, k, n_sink, n_local):
    """The selection among the collected candidates has a short way (fine histogram + bitmap in shared memory: lists of
    up to 8192 and of up to 16384 candidates take different instantiations) and a general way (radix select + counting
    sort: longer lists, sequences whose bitmap does not fit, a split bin with many equal scores).  Normal scores with a
    slice of exact ties right at the threshold; every case must give the oracle's selection."""
    from paper_2609_17652_b200 import binding as fb
    lay = fb.make_layout(1, Hq, n)
    assert fb.fathom_topk_passes(lay, k) == 1
    r = np.random.default_rng(n + k)
    s = np.zeros((Hq, lay.score_stride), dtype=np.float32)
    s[:, :n] = r.standard_normal((Hq, n)).astype(np.float32)
    kth = np.sort(s[Hq - 1, :n])[-k]                             # last head: 40 exact copies of its k-th largest score
    s[Hq - 1, r.choice(n, 40, replace=False)] = kth
    sc = torch.from_numpy(s).cuda()
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    idx = torch.full((Hq, k), -1, dtype=torch.int32, device="cuda")
    for _ in range(2):                                           # scratch and counters reused
        ctx.fathom_topk(lay, sc, k, n_sink, n_local, idx)
    want = O.topk(s[:, :n].astype(np.float64), k, n_sink, n_local)
    assert np.array_equal(idx.cpu().numpy(), want)
    assert ctx.fathom_device_status() == 0
    ctx.close()


def test_topk_narrow_band_of_tied_scores():
    """Scores 5 +- 0.004: a handful of fp32 values per token, all in two bins of the 12-bit histogram, so half of the
    row is a candidate and about eighty tokens share every score.  The list is far too long for shared memory: radix
    passes over global memory, the undecided digit pulled into the cache, its ties decided by the token index."""
    from paper_2609_17652_b200 import binding as fb
    n, Hq, k = 700_000, 3, 4096
    lay = fb.make_layout(1, Hq, n)
    assert fb.fathom_topk_passes(lay, k) == 1
    r = np.random.default_rng(5)
    s = np.zeros((Hq, lay.score_stride), dtype=np.float32)
    s[:, :n] = (r.standard_normal((Hq, n)) * 1e-3 + 5.0).astype(np.float32)
    sc = torch.from_numpy(s).cuda()
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    for n_sink, n_local in ((0, 0), (2, 15)):
        idx = torch.full((Hq, k), -1, dtype=torch.int32, device="cuda")
        ctx.fathom_topk(lay, sc, k, n_sink, n_local, idx)
        assert np.array_equal(idx.cpu().numpy(), O.topk(s[:, :n].astype(np.float64), k, n_sink, n_local))
        assert ctx.fathom_device_status() == 0
    ctx.close()


def test_topk_random_lengths_counts_and_score_distributions():
    """Fifty seeded draws of (n, heads, k, forced tokens, score distribution): normal, rounded (ties), spread growing
    along the row, two-sided exponential, a narrow band far from zero.  Between them they take the two-pass path, the
    short and the general way of the single-pass selection, lists of every length and sequences too long for the
    shared-memory bitmap; draw 49 (1.3 M tokens, k = 16384, narrow band) once lost winners to a list length that was
    read before the list was complete."""
    from paper_2609_17652_b200 import binding as fb
    r = np.random.default_rng(7)
    for it in range(50):
        n = int(r.choice([66000, 70001, 131072, 200003, 262144 + 5, 400000, 1048576, 1300000, 2100000, 2500000]))
        Hq = int(r.choice([1, 2, 3, 5]))
        k = min(int(r.choice([256, 300, 1000, 2048, 4096, 6000, 8192, 16384])), n // 8)
        lay = fb.make_layout(1, Hq, n)
        dist = int(r.integers(0, 5))
        s = np.zeros((Hq, lay.score_stride), dtype=np.float32)
        if dist == 0:
            x = r.standard_normal((Hq, n))
        elif dist == 1:
            x = np.round(r.standard_normal((Hq, n)), 2)
        elif dist == 2:
            x = r.standard_normal((Hq, n)) * np.linspace(0.2, 3, n)[None]
        elif dist == 3:
            x = r.exponential(1.0, (Hq, n)) * r.choice([-1, 1], (Hq, n))
        else:
            x = r.standard_normal((Hq, n)) * 1e-3 + 5.0
        s[:, :n] = x.astype(np.float32)
        n_sink, n_local = (0, 0) if r.random() < 0.5 else (int(r.integers(0, 9)), int(r.integers(0, 70)))
        if n_sink + n_local > k:
            n_sink, n_local = 0, 0
        sc = torch.from_numpy(s).cuda()
        ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
        idx = torch.full((Hq, k), -1, dtype=torch.int32, device="cuda")
        ctx.fathom_topk(lay, sc, k, n_sink, n_local, idx)
        want = O.topk(s[:, :n].astype(np.float64), k, n_sink, n_local)
        assert np.array_equal(idx.cpu().numpy(), want), (it, n, Hq, k, dist, n_sink, n_local)
        assert ctx.fathom_device_status() == 0, it
        ctx.close()
        del sc, idx


def test_topk_at_the_largest_k_on_every_path():
    """k = FATHOM_MAX_K (16384): the direct select then holds 2 x 16384 tokens, the composite cache and the range
    counters in shared memory at once.  Single-pass and two-pass selection and the fused scan + selection."""
    from paper_2609_17652_b200 import binding as fb
    n, Hkv, Hq, k = 540_000 + 11, 1, 2, 16384
    assert fb.fathom_topk_passes(fb.make_layout(Hkv, Hq, n), k) == 1
    L = make_layer(n, Hkv, Hq, seed=33, device="cuda")
    g = run_gpu(L, 48, k, 2, stages=("scan", "topk"))
    ref = O.topk(g["scores"].astype(np.float64), k)
    assert np.array_equal(g["idx"], ref)
    # forced sink / local tokens together with the largest k, on the scores just computed
    lay = fb.make_layout(Hkv, Hq, n)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    sc = torch.zeros((Hq, lay.score_stride), device="cuda"); sc[:, :n] = torch.from_numpy(g["scores"]).cuda()
    idx = torch.empty((Hq, k), dtype=torch.int32, device="cuda")
    ctx.fathom_topk(lay, sc, k, 4, 32, idx)
    assert np.array_equal(idx.cpu().numpy(), O.topk(g["scores"].astype(np.float64), k, 4, 32))
    # fused: same selection without the score array
    planes, scales = g["planes_t"], g["scales_t"]
    depth = torch.from_numpy(g["depth"]).cuda()
    idx2 = torch.empty((Hq, k), dtype=torch.int32, device="cuda")
    ctx.fathom_scan_topk(lay, planes, scales, L.q, depth, 2, k, 0, 0, idx2)
    assert np.array_equal(idx2.cpu().numpy(), ref)
    assert ctx.fathom_device_status() == 0
    ctx.close()


@pytest.mark.parametrize("n,dtype", [(1, torch.float32), (100, torch.float32), (257, torch.float32), (5000, torch.bfloat16),
                                     (8192 + 77, torch.float32), (70000, torch.float32)])
def test_rotated_store_in_one_call_equals_rotate_then_build(n, dtype):
    """fathom_build_planes_rotated gives bit for bit the planes and scales of fathom_rotate_keys followed by
    fathom_build_planes (both of which are checked against the oracle elsewhere), for tiny, ragged and multi-unit
    sequences, three KV heads, fp32 and bf16 keys; a channel of constant keys exercises the zero scale."""
    from paper_2609_17652_b200 import binding as fb
    Hkv, Hq = 3, 6
    g = torch.Generator(device="cuda"); g.manual_seed(2000 + n)
    mix = torch.linalg.qr(torch.randn(Hkv, 128, 128, device="cuda", generator=g))[0]
    sig = torch.exp(torch.rand(Hkv, 1, 128, device="cuda", generator=g) * 3.0 - 2.0)
    K = (torch.bmm(torch.randn(Hkv, n, 128, device="cuda", generator=g) * sig, mix) + 0.75).to(dtype).contiguous()
    lay = fb.make_layout(Hkv, Hq, n)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, 1))
    mean = K.float().mean(dim=1).contiguous()
    V = torch.linalg.qr(torch.randn(Hkv, 128, 128, device="cuda", generator=g))[0].contiguous()
    V[1] = torch.eye(128, device="cuda"); K[1, :, 5] = 3.0; mean[1, 5] = 3.0       # rotated channel 5 of head 1 is all zero
    K_rot = torch.empty((Hkv, n, 128), device="cuda")
    ctx.fathom_rotate_keys(lay, K, mean, V, K_rot)
    nb = (n + 63) // 64
    p_ref = torch.full((Hkv, 128, 4, lay.plane_stride_words), -1, dtype=torch.int64, device="cuda")
    s_ref = torch.full((Hkv, 128, lay.scale_stride), -1, dtype=torch.int16, device="cuda")
    ctx.fathom_build_planes(lay, K_rot, p_ref, s_ref)
    p_one = torch.full_like(p_ref, -1); s_one = torch.full_like(s_ref, -1)
    ctx.fathom_build_planes_rotated(lay, K, mean, V, p_one, s_one)
    ctx.fathom_build_planes_rotated(lay, K, mean, V, p_one, s_one)                 # scratch reuse
    torch.cuda.synchronize()
    assert torch.equal(p_one[..., :nb], p_ref[..., :nb])
    assert torch.equal(s_one[..., :nb], s_ref[..., :nb])
    assert torch.all(p_one[..., nb:] == -1) and torch.all(s_one[..., nb:] == -1)   # padding untouched
    assert torch.all(s_one[1, 5, :nb] == 0) and torch.all(p_one[1, 5, 1:, :nb] == 0)
    assert ctx.fathom_device_status() == 0
    ctx.close()


@pytest.mark.parametrize("hpp,host,ctas", [(4, False, None), (1, False, None), (4, True, None), (4, False, 7), (2, True, 3)])
def test_batched_scan_equals_one_scan_per_session(hpp, host, ctas):
    """fathom_scan_batch over ragged sessions (lengths that are not multiples of 64 or of the 1024-token tile, one of
    a single token) gives bit for bit the scores of one fathom_scan per session, with the planes in HBM or in pinned
    host memory, more sessions than one launch takes (33 > 32), and with so few CTAs that each crosses from one session
    to the next several times."""
    from paper_2609_17652_b200 import binding as fb
    Hkv, Hq = 2, 8
    lengths = [1, 63, 1000, 1024, 1025, 5000, 70001] + [300 + 37 * i for i in range(26)]
    assert len(lengths) == 33
    ctx = fb.Context(0, 1 << 20)
    items, singles = [], []
    for s_i, n in enumerate(lengths):
        L = make_layer(max(n, 64), Hkv, Hq, seed=60, session=s_i, device="cuda")
        K = L.K[:, :n].contiguous()
        lay = fb.make_layout(Hkv, Hq, n)
        planes = torch.zeros((Hkv, 128, 4, lay.plane_stride_words), dtype=torch.int64, device="cuda")
        scales = torch.zeros((Hkv, 128, lay.scale_stride), dtype=torch.int16, device="cuda")
        ctx.fathom_build_planes(lay, K, planes, scales)
        depth = torch.zeros((Hq // hpp, 128), dtype=torch.uint8, device="cuda")
        ctx.fathom_alloc_depth(lay, L.q, L.var, fb.DEPTH_WATERFILL, 48, hpp, depth)
        if host:
            hp = torch.empty(planes.shape, dtype=planes.dtype, pin_memory=True); hp.copy_(planes)
            hs = torch.empty(scales.shape, dtype=scales.dtype, pin_memory=True); hs.copy_(scales)
            planes, scales = hp, hs
        one = torch.full((Hq, lay.score_stride), float("nan"), device="cuda")
        ctx.fathom_scan(lay, planes, scales, L.q, depth, hpp, one)
        many = torch.full((Hq, lay.score_stride), float("nan"), device="cuda")
        items.append((lay, planes, scales, L.q, depth, many))
        singles.append((one, n))
    fb.fathom_scan_set_ctas_per_plan(ctas or 0)         # few CTAs per plan: each walks tiles of several sessions in turn
    try:
        ctx.fathom_scan_batch(items, hpp)
        torch.cuda.synchronize()
    finally:
        fb.fathom_scan_set_ctas_per_plan(0)
    for (lay, _, _, _, _, many), (one, n) in zip(items, singles):
        assert torch.equal(many[:, :n], one[:, :n])
        assert torch.isnan(many[:, n:]).all()                                # padding untouched
    assert ctx.fathom_device_status() == 0
    ctx.close()


def test_single_pass_calibration_with_drifting_and_outlying_keys():
    """The one-read covariance centres the keys on a shift taken from 64 keys spread over the sequence.  Keys whose mean
    drifts along the sequence, with a few far-off keys at the start (as the first tokens of a prompt often are), must
    still give the oracle's mean and covariance: nothing may cancel."""
    from paper_2609_17652_b200 import binding as fb
    Hkv, Hq, n = 2, 4, 30000
    g = torch.Generator(device="cuda"); g.manual_seed(99)
    K = torch.randn(Hkv, n, 128, device="cuda", generator=g)
    K += torch.linspace(-4.0, 6.0, n, device="cuda")[None, :, None] * torch.rand(Hkv, 1, 128, device="cuda", generator=g)   # drift
    K[:, :4] += 80.0                                                              # outlying first keys
    K = K.contiguous()
    lay = fb.make_layout(Hkv, Hq, n)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, 1))
    mean = torch.zeros((Hkv, 128), device="cuda"); cov = torch.zeros((Hkv, 128, 128), device="cuda")
    var = torch.zeros((Hkv, 128), device="cuda")
    ctx.fathom_channel_variance(lay, K, mean, var)
    mu_v, var_ref = O.channel_variance(K.cpu().numpy())
    assert np.all(np.abs(mean.cpu().numpy() - mu_v) <= 1e-6 * np.abs(mu_v) + 1e-5 * np.sqrt(var_ref))
    assert np.all(np.abs(var.cpu().numpy() - var_ref) <= 1e-5 * var_ref)
    ctx.fathom_calibrate(lay, K, mean, cov)
    mu_ref, C_ref = O.calibrate(K.cpu().numpy())
    assert np.allclose(mean.cpu().numpy(), mu_ref, rtol=1e-5, atol=1e-5)
    scale = np.abs(C_ref).max(axis=(1, 2), keepdims=True)
    assert np.all(np.abs(cov.cpu().numpy() - C_ref) <= 2e-5 * scale)
    ctx.close()


def test_per_layer_budgets_closed_on_synthetic_layers():
    """Sec. 3.4 end to end: the error of every synthetic layer at every level measured through the library, the greedy plan
    of fathom_plan_layer_budgets (equal to the oracle's on the same table), and the planned budgets passed through
    fathom_alloc_depth: the granted depths of layer l sum to its planned budget, and the budgets stay within the target."""
    import bench
    from paper_2609_17652_b200 import binding as fb
    n, Hkv, Hq, k, hpp, nl, target = 20000, 2, 8, 256, 4, 5, 48.0
    levels = [24, 32, 48, 64, 96]
    lay = fb.make_layout(Hkv, Hq, n)
    ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
    Ls = [make_layer(n, Hkv, Hq, seed=6, layer=l, device="cuda", **bench.layer_recipe(l)) for l in range(nl)]
    err, bits, sums = bench.measure_layer_errors(fb, ctx, lay, Ls, levels, k, hpp, torch.cuda.current_stream())
    assert ctx.fathom_device_status() == 0
    choice = fb.fathom_plan_layer_budgets(err, levels, target)
    assert choice == list(O.plan_layer_budgets(np.array(err), levels, target))
    planned = [levels[c] for c in choice]
    assert sum(planned) <= target * nl
    # no single raise still fits that would lower the error: the plan is not trivially stuck at the lowest level
    assert sum(planned) > levels[0] * nl
    depth = torch.zeros((Hq // hpp, 128), dtype=torch.uint8, device="cuda")
    for l, L in enumerate(Ls):
        ctx.fathom_alloc_depth(lay, L.q, L.var, fb.DEPTH_WATERFILL, planned[l], hpp, depth)
        torch.cuda.synchronize()
        assert np.all(depth.cpu().numpy().sum(1) == planned[l])
        assert sums[l][choice[l]] == [planned[l]] * (Hq // hpp)
    for l in range(nl):                                                        # more bits are read at higher levels
        assert all(b1 > b0 for b0, b1 in zip(bits[l], bits[l][1:]))
    ctx.close()

"""The allocation-free attention entry point (for callers that were only handed buffers and cannot ask the
driver for device memory) must give what the context-based entry point gives.  Collected last on purpose."""
import math

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(seed, n, Hkv, Hq, k):
    g = torch.Generator(device="cuda").manual_seed(seed)
    q = torch.randn(Hq, 128, generator=g, device="cuda")
    Kr = torch.randn(Hkv, n, 128, generator=g, device="cuda").to(torch.bfloat16)
    Vr = torch.randn(Hkv, n, 128, generator=g, device="cuda").to(torch.bfloat16)
    idx = torch.stack([torch.randperm(n, generator=g, device="cuda")[:k].sort().values for _ in range(Hq)]).to(torch.int32)
    return q, Kr, Vr, idx


def test_static_entry_matches_context_entry_on_two_calls_in_a_row():
    from paper_2609_17652_b200 import binding as fb
    n, Hkv, Hq = 6000, 2, 8
    lay = fb.make_layout(Hkv, Hq, n)
    scale = 1.0 / math.sqrt(128)
    # second call is smaller than the first: stale partials of the first call lie beyond what it uses
    for call, (seed, k) in enumerate([(1, 700), (2, 130)]):
        q, Kr, Vr, idx = _case(seed, n, Hkv, Hq, k)
        ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
        want = torch.full((Hq, 128), float("nan"), device="cuda")
        ctx.fathom_sparse_attend(lay, q, Kr, Vr, idx, k, scale, want)
        got = torch.full((Hq, 128), float("nan"), device="cuda")
        fb.fathom_sparse_attend_static(lay, q, Kr, Vr, idx, k, scale, got)
        torch.cuda.synchronize()
        ctx.close()
        w, g = want.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(g)), call
        rel = np.linalg.norm(g - w, axis=1) / np.linalg.norm(w, axis=1)
        assert rel.max() <= 2e-3, (call, rel.max())          # the tolerance of the attention parity tests
        assert np.array_equal(g, w), call                     # same kernels, same order: in fact identical


def test_static_entry_at_its_limit_then_a_small_call_with_fp32_rows():
    """Exactly FATHOM_ATTEND_STATIC_MAX_CHUNKS chunks (32 heads x ceil(8192 / 128) = 2048: the last element of the built-in
    array is used), then a much smaller call with fp32 rows: both bit for bit what the context-based entry point gives."""
    from paper_2609_17652_b200 import binding as fb
    scale = 1.0 / math.sqrt(128)
    for call, (seed, n, Hkv, Hq, k, f32) in enumerate([(5, 9000, 8, 32, 8192, False), (6, 3000, 2, 8, 200, True)]):
        assert Hq * ((k + 127) // 128) <= fb.ATTEND_STATIC_MAX_CHUNKS
        lay = fb.make_layout(Hkv, Hq, n)
        q, Kr, Vr, idx = _case(seed, n, Hkv, Hq, k)
        if f32:
            Kr, Vr = Kr.float(), Vr.float()
        ctx = fb.Context(0, fb.fathom_scratch_bytes(lay, k))
        want = torch.full((Hq, 128), float("nan"), device="cuda")
        ctx.fathom_sparse_attend(lay, q, Kr, Vr, idx, k, scale, want)
        got = torch.full((Hq, 128), float("nan"), device="cuda")
        fb.fathom_sparse_attend_static(lay, q, Kr, Vr, idx, k, scale, got)
        torch.cuda.synchronize()
        ctx.close()
        assert torch.isfinite(got).all(), call
        assert torch.equal(got, want), call


def test_static_entry_rejects_sizes_beyond_its_built_in_scratch():
    from paper_2609_17652_b200 import binding as fb
    lay = fb.make_layout(8, 32, 20000)
    x = torch.zeros(4096, device="cuda")
    with pytest.raises(fb.FathomError) as e:                  # 32 heads * ceil(16384 / 128) = 4096 chunks > 2048
        fb.fathom_sparse_attend_static(lay, x, x, x, x, 16384, 1.0, x, row_dtype=fb.BF16)
    assert e.value.status == -6 and "built-in" in str(e.value)
    fb.lib.fathom_strerror(-6)

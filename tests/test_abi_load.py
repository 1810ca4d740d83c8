"""No-GPU checks of the boundary: the shared library loads, exports every symbol the header declares,
and rejects bad arguments on the host before any launch."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def fb():
    from paper_2609_17652_b200 import build
    build.build()
    from paper_2609_17652_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fathom.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fathom_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(fb):
    names = declared_functions()
    assert len(names) >= 12 and {"fathom_build_planes", "fathom_alloc_depth", "fathom_scan", "fathom_topk",
                                 "fathom_sparse_attend"} <= set(names)
    for name in names:
        assert hasattr(fb.lib, name), name
    assert set(fb.EXPORTS) == set(names)


def test_version_and_error_text(fb):
    assert fb.fathom_version() >= 100
    for code in range(0, -6, -1):
        assert len(fb.lib.fathom_strerror(code)) > 1
    assert b"unknown" in fb.lib.fathom_strerror(-99)


def test_layout_struct_matches_header(fb):
    assert C.sizeof(fb.Layout) == 4 * 4 + 4 * 8
    lay = fb.make_layout(8, 32, 1 << 20)
    assert lay.plane_stride_words == 16384 and lay.scale_stride == 16384 and lay.score_stride == 1 << 20
    odd = fb.make_layout(1, 1, 65, row_align_bytes=16)              # the tightest strides the layout allows
    assert odd.plane_stride_words == 2 and odd.scale_stride == 8 and odd.score_stride == 68
    odd = fb.make_layout(1, 1, 65)                                  # default: every row starts on a 128-byte boundary
    assert odd.plane_stride_words == 16 and odd.scale_stride == 64 and odd.score_stride == 96


def test_scratch_bytes_and_host_side_rejection(fb):
    lay = fb.make_layout(8, 32, 1 << 20)
    need = fb.fathom_scratch_bytes(lay, 4096)
    assert need >= 32 * (1 << 20) * 4                      # candidate list can hold every token
    bad = fb.make_layout(8, 32, 1 << 20); bad.d = 64
    assert fb.fathom_scratch_bytes(bad, 4096) == 0
    bad = fb.make_layout(8, 32, 1 << 20); bad.n_q_heads = 30
    assert fb.fathom_scratch_bytes(bad, 4096) == 0
    # a NULL context is refused before anything touches a device
    assert fb.lib.fathom_scan(None, C.byref(lay), 16, 16, 16, 16, 4, 16, None) == -1
    assert fb.lib.fathom_topk(None, C.byref(lay), 16, 10, 0, 0, 16, None) == -1
    assert fb.lib.fathom_build_planes(None, C.byref(lay), 16, 0, 16, 16, None) == -1
    assert fb.lib.fathom_alloc_depth(None, C.byref(lay), 16, 16, 0, 48, 4, 16, None) == -1
    assert fb.lib.fathom_sparse_attend(None, C.byref(lay), 16, 16, 16, 1, 16, 10, C.c_float(1.0), 16, None) == -1
    assert fb.lib.fathom_destroy(None) == 0


def test_layer_budget_plan_host_function_matches_the_oracle(fb):
    """fathom_plan_layer_budgets is host code: compared here, level by level, with the oracle's greedy plan on random
    error tables (convex and not), uneven level spacing, ties and targets between two sums."""
    import numpy as np
    from oracle import fathom_oracle as O
    r = np.random.default_rng(5)
    for trial in range(60):
        L = int(r.integers(1, 40)); nlev = int(r.integers(1, 9))
        levels = np.cumsum(r.integers(1, 17, size=nlev)) + 16
        err = r.uniform(0, 1, size=(L, nlev))
        if trial % 3 == 0:
            err = -np.sort(-err, axis=1)                   # falling curves
        if trial % 4 == 0:
            err = np.round(err, 1)                         # many ties
        target = float(r.uniform(levels[0] - 1, levels[-1] + 1))
        got = fb.fathom_plan_layer_budgets(err.tolist(), levels.tolist(), target)
        ref = O.plan_layer_budgets(err, levels, target)
        assert got == list(ref), (trial, L, nlev, target)
        assert sum(levels[i] for i in got) <= max(target, levels[0]) * L + 1e-9
    # the paper's range at its two means: 36 layers, levels 24 .. 128 in steps of 8
    levels = list(range(24, 129, 8))
    err = np.exp(-np.outer(r.uniform(0.01, 0.06, 36), levels))
    for mean in (48, 64):
        got = fb.fathom_plan_layer_budgets(err.tolist(), levels, mean)
        assert got == list(O.plan_layer_budgets(err, levels, mean))
        assert sum(levels[i] for i in got) == mean * 36
    assert fb.lib.fathom_plan_layer_budgets(None, 1, 1, None, C.c_double(1.0), None) == -1
    bad = (C.c_int * 2)(32, 32); e = (C.c_double * 2)(1.0, 0.5); out = (C.c_int * 1)()
    assert fb.lib.fathom_plan_layer_budgets(e, 1, 2, bad, C.c_double(40.0), out) == -1


def test_topk_pass_plan_and_rejections_of_the_newer_entry_points(fb):
    """Host logic only: which rows fathom_topk reads once, and NULL / inconsistent arguments of the entry points
    beyond the five calls are refused before any launch."""
    lay = fb.make_layout(8, 32, 1 << 20)
    assert fb.fathom_topk_passes(lay, 4096) == 1 and fb.fathom_topk_passes(lay, 4096, 4, 32) == 1
    assert fb.fathom_topk_passes(lay, 64) == 2                       # too few winners to estimate from a sample
    assert fb.fathom_topk_passes(fb.make_layout(8, 32, 40000), 2048) == 2     # too short to sample
    assert fb.fathom_topk_passes(fb.make_layout(8, 32, 131072), 2048) == 1
    assert fb.lib.fathom_topk_passes(C.byref(lay), 0, 0, 0) < 0 and fb.lib.fathom_topk_passes(C.byref(lay), 10, 8, 8) < 0
    for call, nargs in (("fathom_scan_topk", 12), ("fathom_gather_union", 12), ("fathom_calibrate", 7), ("fathom_rotate_keys", 8),
                        ("fathom_rotate_query", 6), ("fathom_channel_variance", 7), ("fathom_build_planes_rotated", 9)):
        fn = getattr(fb.lib, call)
        args = [None, C.byref(lay)] + [16] * (nargs - 2)
        if call in ("fathom_calibrate", "fathom_rotate_keys", "fathom_channel_variance", "fathom_build_planes_rotated"):
            args[3] = 0                                              # k_dtype
        if call == "fathom_scan_topk":
            args[6:10] = [4, 10, 0, 0]
        if call == "fathom_gather_union":
            args[3] = 10; args[6] = 1
        args[-1] = None                                              # stream
        assert fn(*args) == -1, call                                 # FATHOM_ERR_INVALID_ARG: NULL context
    assert fb.lib.fathom_scan_batch(None, None, 1, 4, None) == -1

"""Pins the oracle to the numbers the paper prints in its Appendix A worked example."""
import json
import os

import numpy as np
import pytest

from oracle import fathom_oracle as O


@pytest.fixture(scope="module")
def ex(golden_dir):
    with open(os.path.join(golden_dir, "appendix_a_worked_example.json")) as f:
        return json.load(f)


def _inputs(ex):
    K = np.array(ex["K"], dtype=np.float32)[None]              # [1][6][4]
    q = np.array([ex["q_head_A"], ex["q_head_B"]], dtype=np.float32)
    return K, q


def test_variance_convention_is_unbiased(ex):
    K, _ = _inputs(ex)
    v = K[0].astype(np.float64).var(axis=0, ddof=1)
    # first three printed values to 3 decimals; the 4th prints as 0.001 (0.0015 unrounded)
    assert np.allclose(v[:3], ex["var_printed"][:3], atol=6e-4)
    assert abs(v[3] - ex["var_printed"][3]) < 6e-4
    assert not np.allclose(K[0].astype(np.float64).var(axis=0, ddof=0)[:3], ex["var_printed"][:3], atol=6e-4)


def test_importance_matches_printed_g(ex):
    _, q = _inputs(ex)
    var = np.array([ex["var_printed"]], dtype=np.float32)
    g = O.importance(q, var, heads_per_plan=2)[0]
    assert np.allclose(g, ex["g_printed"], atol=6e-3)
    # per-head importance would not: the printed g needs the sum over the group
    g1 = O.importance(q, np.repeat(var, 1, 0), heads_per_plan=1)
    assert not np.allclose(g1[0], ex["g_printed"], atol=6e-3)


def test_bisection_trace_and_depths(ex):
    _, q = _inputs(ex)
    var = np.array([ex["var_printed"]], dtype=np.float32)
    g = O.importance(q, var, 2)[0]
    bis = ex["bisection_B8"]
    t, theta, trace = O.waterfill_depths_bisection(g, 8, *bis["bracket"], steps=30)
    for row, (lo, hi, mid, tt, s) in zip(bis["rows"], trace):
        assert abs(mid - row["trial"]) <= 0.006 * row["trial"] + 1e-4
        assert list(tt) == row["t"] and s == row["sum"] and (s <= 8) == row["fits"]
        x = np.log(g[:3] / mid) / np.log(4.0)
        assert np.allclose(x, row["log4"][:3], atol=0.011)
    assert abs(theta - bis["theta_after_30"]) < 6e-4
    assert list(t) == bis["depths"]
    # the exact sorted-priority rule gives the same plans at both budgets
    assert list(O.waterfill_depths(g, 8)) == bis["depths"]
    assert list(O.waterfill_depths(g, 6)) == ex["B6"]["depths"]
    t6, theta6, _ = O.waterfill_depths_bisection(g, 6, *bis["bracket"], steps=30)
    assert list(t6) == ex["B6"]["depths"] and abs(theta6 - ex["B6"]["theta"]) < 6e-4


def test_channel2_codes_and_one_plane(ex):
    K, _ = _inputs(ex)
    codes, scales = O.quantise_block_codes(K)
    assert float(scales[0, 2, 0]) == ex["channel2"]["cell_width"]
    assert list(codes[0, :, 2]) == ex["channel2"]["codes"]
    planes = O.pack_planes(codes)
    v = O.prefix_values(planes, scales, 6, 0, 2, 1)
    assert np.allclose(v, ex["channel2"]["one_plane_values"], atol=0)
    # the sign plane is the MSB of the printed codes
    assert int(planes[0, 2, 0, 0]) == sum(((c >> 3) & 1) << i for i, c in enumerate(ex["channel2"]["codes"]))


def test_scale_is_rounded_before_quantising(ex):
    """Key t1, channel 1: 0.9 / (1.2/8) sits on a cell edge; only the stored fp16 scale
    (0.15002...) gives code 13 and the printed approximate scores."""
    K, _ = _inputs(ex)
    codes, scales = O.quantise_block_codes(K)
    assert codes[0, 1, 1] == 13
    assert float(scales[0, 1, 0]) > 0.15


def test_approximate_and_exact_scores(ex):
    K, q = _inputs(ex)
    planes, scales = O.build_planes(K)
    depth = np.array([ex["bisection_B8"]["depths"]], dtype=np.uint8)
    s = O.scan(planes, scales, q, depth, 6, heads_per_plan=2)
    assert np.allclose(s[0], ex["depths_4310"]["approx_scores_A"], atol=6e-3)
    assert np.allclose(s[1], ex["depths_4310"]["approx_scores_B"], atol=6e-3)
    s2 = O.scan_signed_planes(planes, scales, q, depth, 6, 2)
    assert np.allclose(s, s2, rtol=0, atol=1e-12)
    e = O.exact_scores(q, K)
    assert np.allclose(e[0], ex["depths_4310"]["exact_scores_A"], atol=6e-3)
    assert np.allclose(e[1], ex["depths_4310"]["exact_scores_B"], atol=6e-3)


def test_top2_sets_and_failure_at_B6(ex):
    K, q = _inputs(ex)
    planes, scales = O.build_planes(K)
    d8 = np.array([ex["bisection_B8"]["depths"]], dtype=np.uint8)
    idx = O.topk(O.scan(planes, scales, q, d8, 6, 2), 2)
    assert list(idx[0]) == ex["depths_4310"]["top2_A"] and list(idx[1]) == ex["depths_4310"]["top2_B"]
    assert list(O.topk(O.exact_scores(q, K), 2)[1]) == ex["depths_4310"]["top2_B"]
    d6 = np.array([ex["B6"]["depths"]], dtype=np.uint8)
    idx6 = O.topk(O.scan(planes, scales, q, d6, 6, 2), 2)
    assert list(idx6[1]) == ex["B6_top2_B_wrong"]


def test_fixed_channel_rule(ex):
    K, q = _inputs(ex)
    dep = O.fixed_channel_depths(q, heads_per_plan=2, r=2)
    assert [j for j in range(4) if dep[0, j] == 4] == ex["sparq_r2"]["channels"]
    assert np.allclose(np.abs(q.astype(np.float64)).sum(0), ex["sparq_r2"]["sum_abs_q"], atol=1e-6)
    planes, scales = O.build_planes(K)
    idx = O.topk(O.scan(planes, scales, q, dep, 6, 2), 2)
    assert list(idx[1]) == ex["sparq_r2"]["top2_B"]

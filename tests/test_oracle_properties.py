"""Pins the oracle to closed forms, invariants and brute force (no GPU)."""
import itertools
from fractions import Fraction

import numpy as np
import pytest

from oracle import fathom_oracle as O


def rng_keys(seed, Hkv, n, d, scale=1.0):
    r = np.random.default_rng(seed)
    sig = np.exp(r.uniform(np.log(0.1), np.log(4.0), size=(Hkv, 1, d)))
    return (r.standard_normal((Hkv, n, d)) * sig * scale).astype(np.float32)


# ---------------------------------------------------------------- O1 codes / planes
@pytest.mark.parametrize("n", [1, 63, 64, 65, 127, 200])
def test_codes_match_exact_rational_floor(n):
    """Brute force with exact rationals: code = clip(floor(k / S), -8, 7) + 8 with S the
    stored fp16 scale of the block (Eq. 2); tail block uses the real tokens only."""
    K = rng_keys(n, 2, n, 5)
    K[0, 0, 0] = 0.0
    if n > 3:
        K[1, :, 3] = 0.0                                     # an all-zero channel -> scale 0 -> code 8
    codes, scales = O.quantise_block_codes(K)
    for h in range(2):
        for j in range(5):
            for b in range((n + 63) // 64):
                blk = K[h, b * 64:(b + 1) * 64, j]
                a = max(abs(Fraction(float(x))) for x in blk)
                S = np.float16(np.float32(float(a / 8)))
                assert scales[h, j, b] == S
                for r, x in enumerate(blk):
                    if float(S) == 0.0:
                        want = 8
                    else:
                        fl = Fraction(float(x)) / Fraction(float(S))
                        want = min(max(fl.numerator // fl.denominator, -8), 7) + 8
                    assert codes[h, b * 64 + r, j] == want


def test_cell_edge_cases():
    """k exactly on a cell edge m*S lands in cell m; k = +a clips to 7; k = -a gives 0."""
    S = np.float32(np.float16(0.3))
    col = np.array([m * float(S) for m in range(-8, 9)], dtype=np.float32)     # exact products
    K = col.reshape(1, -1, 1)
    codes, scales = O.quantise_block_codes(K)
    assert float(scales[0, 0, 0]) == float(S)
    assert list(codes[0, :, 0]) == [0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15, 15]
    below = np.nextafter(col, np.float32(-np.inf))
    below[0] = col[0]; below[-1] = col[-1]                   # keep the block max unchanged
    codes2, _ = O.quantise_block_codes(below.reshape(1, -1, 1))
    assert list(codes2[0, 1:-1, 0]) == list(range(0, 15))


def test_dequantised_value_is_within_one_cell():
    K = rng_keys(3, 2, 300, 16)
    codes, scales = O.quantise_block_codes(K)
    S = np.repeat(scales.astype(np.float64), 64, axis=2)[:, :, :300].transpose(0, 2, 1)
    err = np.abs((codes.astype(np.float64) - 7.5) * S - K)
    top, bot = codes == 15, codes == 0
    mid = ~top & ~bot
    assert np.all(err[mid] <= S[mid] / 2 + 1e-12)
    # -a can fall just outside cell -8 when fp16 rounding shrinks the scale (8 * 2^-11 of a cell)
    assert np.all(err[bot] <= S[bot] / 2 * (1 + 0.01) + 1e-12)
    assert np.all(err[top] <= S[top] * (1 + 0.01) + 1e-12)   # the +a clip may be a full cell off


@pytest.mark.parametrize("n", [1, 64, 65, 130])
def test_plane_packing_loop_equals_vectorised_and_roundtrips(n):
    K = rng_keys(10 + n, 2, n, 7)
    codes, _ = O.quantise_block_codes(K)
    p1, p2 = O.pack_planes(codes), O.pack_planes_fast(codes)
    assert p1.dtype == np.uint64 and np.array_equal(p1, p2)
    back = O.unpack_codes(p1, n, 4)                          # decoding all 4 planes returns c
    assert np.array_equal(back.transpose(0, 2, 1), codes)
    # bits of absent tail tokens are zero
    if n % 64:
        assert np.all(p1[..., -1] >> np.uint64(n % 64) == 0)


def test_store_is_68_bytes_per_token():
    K = rng_keys(0, 1, 64 * 10, 128)
    planes, scales = O.build_planes(K)
    assert (planes.nbytes + scales.nbytes) / (64 * 10) == 68.0


@pytest.mark.parametrize("t", [1, 2, 3, 4])
def test_prefix_is_the_t_bit_midrise_quantiser(t):
    """Independent path: quantise k directly with 2^t cells of width a/2^(t-1) over [-a, a)
    (a = 8 S), exact rationals, and compare with c >> (4 - t) and with the dequantised value."""
    n, d = 150, 6
    K = rng_keys(40 + t, 1, n, d)
    planes, scales = O.build_planes(K)
    ct = O.unpack_codes(planes, n, t)
    for j in range(d):
        vals = O.prefix_values(planes, scales, n, 0, j, t)
        for i in range(n):
            S = Fraction(float(scales[0, j, i // 64]))
            a = 8 * S
            w = a / 2 ** (t - 1)
            if S == 0:
                cell = 0
            else:
                fl = Fraction(float(K[0, i, j])) / w
                cell = min(max(fl.numerator // fl.denominator, -2 ** (t - 1)), 2 ** (t - 1) - 1)
            assert ct[0, j, i] == cell + 2 ** (t - 1)
            assert vals[i] == float((cell + Fraction(1, 2)) * w)


def test_error_variance_falls_about_4x_per_plane():
    r = np.random.default_rng(5)
    K = r.uniform(-1, 1, size=(1, 64 * 200, 8)).astype(np.float32)
    planes, scales = O.build_planes(K)
    mse = []
    for t in range(1, 5):
        v = np.stack([O.prefix_values(planes, scales, K.shape[1], 0, j, t) for j in range(8)], 1)
        mse.append(np.mean((v - K[0]) ** 2))
    ratios = np.array(mse[:-1]) / np.array(mse[1:])
    assert np.all(np.abs(ratios - 4.0) < 0.4)


# ---------------------------------------------------------------- O2 depths
def brute_force_depths(g, B):
    best, arg = None, None
    for t in itertools.product(range(5), repeat=len(g)):
        if sum(t) > B:
            continue
        cost = sum(gj * 4.0 ** (-tj) for gj, tj in zip(g, t))
        if best is None or cost < best - 1e-15 * abs(best):
            best, arg = cost, t
    return best, arg


@pytest.mark.parametrize("seed", range(6))
def test_waterfill_is_the_brute_force_optimum(seed):
    r = np.random.default_rng(seed)
    d = 5
    g = np.exp(r.uniform(np.log(1e-3), np.log(50), size=d))
    for B in [0, 1, 3, 6, 9, 13, 19, 20, 25]:
        t = O.waterfill_depths(g, B)
        assert t.sum() == min(B, 4 * d)
        best, _ = brute_force_depths(g, B)
        cost = float(np.sum(g * 4.0 ** (-t.astype(np.float64))))
        assert cost <= best * (1 + 1e-12)


def test_waterfill_invariants():
    r = np.random.default_rng(11)
    g = np.exp(r.uniform(np.log(1e-4), np.log(100), size=128))
    prev = np.zeros(128, dtype=np.int64)
    for B in [0, 1, 32, 40, 48, 64, 80, 136, 300, 511, 512, 600]:
        t = O.waterfill_depths(g, B).astype(np.int64)
        assert t.sum() == min(B, 512) and t.max() <= 4
        assert np.all(t >= prev)                              # raising B never lowers a depth
        order = np.argsort(-g)
        assert np.all(np.diff(t[order]) <= 0)                 # depth non-increasing in rank of g
        prev = t
    assert np.all(O.waterfill_depths(np.zeros(128), 512) == 4)       # g = 0 still fills at B = 4d
    assert list(O.waterfill_depths(np.array([1.0, 1.0, 1.0]), 2)) == [1, 1, 0]   # ties -> lower channel


def test_waterfill_tie_between_channel_and_plane():
    # g0 4^-2 == g1 4^-1 : lower channel first
    assert list(O.waterfill_depths(np.array([4.0, 1.0]), 2)) == [2, 0]
    # priorities: ch0: .25 .0625 ; ch1: 1 .25 -> sorted: (1,ch1), (.25,ch0), (.25,ch1) ...
    assert list(O.waterfill_depths(np.array([1.0, 4.0]), 2)) == [1, 1]


@pytest.mark.parametrize("seed", range(5))
def test_literal_bisection_agrees_away_from_ties(seed):
    r = np.random.default_rng(100 + seed)
    g = np.exp(r.uniform(np.log(1e-3), np.log(100), size=128))
    pri = np.sort(np.concatenate([g * 4.0 ** (-m) for m in range(1, 5)]))[::-1]
    for B in [32, 48, 80, 136]:
        if pri[B - 1] / pri[B] < 1 + 1e-6:                    # cut sits on a near-tie: skip
            continue
        t, _, _ = O.waterfill_depths_bisection(g, B, 1e-9, 1e4, steps=60)
        assert np.array_equal(t, O.waterfill_depths(g, B))


def test_bits_per_token_convention():
    """Sec. 4 byte accounting: 136 for 32 channels at 4 bits, 68 for 16, 288 for the 2-bit
    thumbnail, 544 for the full 4-bit scan."""
    def row(nch, t):
        x = np.zeros(128, dtype=np.uint8); x[:nch] = t; return x
    assert O.bits_per_token(row(32, 4)) == 136
    assert O.bits_per_token(row(16, 4)) == 68
    assert O.bits_per_token(row(128, 2)) == 288
    assert O.bits_per_token(row(128, 4)) == 544


# ---------------------------------------------------------------- O3 scan
def test_all_planes_scan_is_the_dense_4bit_dot_product():
    Hkv, G, n, d = 2, 2, 333, 128
    K = rng_keys(7, Hkv, n, d)
    q = np.random.default_rng(8).standard_normal((Hkv * G, d)).astype(np.float32)
    codes, scales = O.quantise_block_codes(K)
    planes = O.pack_planes_fast(codes)
    depth = np.full((Hkv, d), 4, dtype=np.uint8)
    s = O.scan(planes, scales, q, depth, n, heads_per_plan=G)
    S = np.repeat(scales.astype(np.float64), 64, axis=2)[:, :, :n].transpose(0, 2, 1)
    deq = (codes.astype(np.float64) - 7.5) * S                # (c - 8 + 1/2) s
    for h in range(Hkv * G):
        ref = deq[h // G] @ q[h].astype(np.float64)
        assert np.allclose(s[h], ref, rtol=1e-12, atol=1e-12)


def test_scan_formulations_and_sampled_tokens_agree():
    Hkv, G, n, d = 2, 4, 500, 128
    K = rng_keys(17, Hkv, n, d)
    r = np.random.default_rng(18)
    q = r.standard_normal((Hkv * G, d)).astype(np.float32)
    var = K.astype(np.float64).var(axis=1, ddof=1).astype(np.float32)
    planes, scales = O.build_planes(K)
    for hpp in (G, 1):
        depth = O.alloc_depth(q, var, "waterfill", 48, hpp)
        a = O.scan(planes, scales, q, depth, n, hpp)
        b = O.scan_signed_planes(planes, scales, q, depth, n, hpp)
        assert np.allclose(a, b, rtol=1e-12, atol=1e-12)
        tok = [0, 1, 63, 64, 65, 257, 499]
        for h in (0, 3, 7):
            assert np.allclose(O.scan_tokens(planes, scales, q, depth, hpp, h, tok), a[h, tok], rtol=1e-13, atol=1e-13)


def test_zero_depth_plan_gives_zero_scores_and_uniform_two_is_the_thumbnail():
    K = rng_keys(21, 1, 100, 128)
    q = np.random.default_rng(22).standard_normal((1, 128)).astype(np.float32)
    planes, scales = O.build_planes(K)
    assert np.all(O.scan(planes, scales, q, np.zeros((1, 128), np.uint8), 100, 1) == 0)
    dep = O.alloc_depth(q, np.ones((1, 128), np.float32), "uniform", 2, 1)
    s = O.scan(planes, scales, q, dep, 100, 1)
    codes, _ = O.quantise_block_codes(K)
    S = np.repeat(scales.astype(np.float64), 64, axis=2)[:, :, :100].transpose(0, 2, 1)
    two_bit = ((codes >> 2).astype(np.float64) + 0.5 - 2.0) * (8 * S) / 2.0
    assert np.allclose(s[0], two_bit[0] @ q[0].astype(np.float64), rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- O4 top-k
def brute_topk(s, k, n_sink, n_local):
    n = len(s)
    forced = set(range(min(n_sink, n))) | set(range(max(0, n - n_local), n))
    rest = [i for i in range(n) if i not in forced]
    rest.sort(key=lambda i: (-(s[i] + 0.0), i))
    return sorted(forced | set(rest[:k - len(forced)]))


@pytest.mark.parametrize("seed", range(4))
def test_topk_matches_python_sort_with_ties(seed):
    r = np.random.default_rng(seed)
    n = 300
    s = np.round(r.standard_normal((3, n)), 1)                # many exact ties
    s[0, 5] = -0.0; s[0, 9] = 0.0
    for k, ns, nl in [(1, 0, 0), (10, 0, 0), (40, 4, 32), (300, 0, 0), (36, 4, 32), (50, 0, 7)]:
        got = O.topk(s, k, ns, nl)
        for h in range(3):
            assert list(got[h]) == brute_topk(list(s[h]), k, ns, nl)


def test_topk_ties_go_to_lower_index_and_signed_zero():
    s = np.array([[1.0, 2.0, 2.0, 2.0, 0.5]])
    assert list(O.topk(s, 2)[0]) == [1, 2]
    z = np.array([[-0.0, 0.0, -0.0, 0.0]])
    assert list(O.topk(z, 2)[0]) == [0, 1]


# ---------------------------------------------------------------- O5 attention
def test_attention_special_cases():
    r = np.random.default_rng(3)
    Hkv, G, n, d = 2, 2, 40, 16
    Kr = r.standard_normal((Hkv, n, d)).astype(np.float32)
    Vr = r.standard_normal((Hkv, n, d)).astype(np.float32)
    q = r.standard_normal((Hkv * G, d)).astype(np.float32)
    sc = 1 / np.sqrt(d)
    # k = n: textbook dense softmax attention in extended precision
    dense = O.dense_attention(q, Kr, Vr, sc)
    for h in range(Hkv * G):
        e = (Kr[h // G].astype(np.longdouble) @ q[h].astype(np.longdouble)) * np.longdouble(sc)
        w = np.exp(e) / np.exp(e).sum()
        assert np.allclose(dense[h], (w @ Vr[h // G].astype(np.longdouble)).astype(np.float64), rtol=1e-12, atol=1e-13)
    # k = 1 returns that V row
    idx = np.array([[7], [0], [39], [11]], dtype=np.int32)
    one = O.sparse_attend(q, Kr, Vr, idx, sc)
    for h in range(4):
        assert np.allclose(one[h], Vr[h // G, idx[h, 0]], rtol=0, atol=1e-15)
    # order of the index list is irrelevant; a constant logit shift (scale 0 -> uniform) gives the mean
    idx2 = np.stack([r.permutation(n)[:9] for _ in range(4)]).astype(np.int32)
    a = O.sparse_attend(q, Kr, Vr, idx2, sc)
    b = O.sparse_attend(q, Kr, Vr, idx2[:, ::-1], sc)
    assert np.allclose(a, b, rtol=1e-13, atol=1e-14)
    u = O.sparse_attend(q, Kr, Vr, idx2, 0.0)
    for h in range(4):
        assert np.allclose(u[h], Vr[h // G, idx2[h]].astype(np.float64).mean(0), rtol=1e-13, atol=1e-14)


def test_attention_is_invariant_to_a_logit_shift():
    """softmax((q + c u) K^T) with K rows all having the same component along u shifts every
    logit by a constant and must not change the output."""
    r = np.random.default_rng(4)
    n, d = 30, 8
    Kr = r.standard_normal((1, n, d)).astype(np.float32)
    Kr[0, :, 0] = 1.0
    Vr = r.standard_normal((1, n, d)).astype(np.float32)
    q = r.standard_normal((1, d)).astype(np.float32)
    q2 = q.copy(); q2[0, 0] += 3.0
    idx = np.arange(n, dtype=np.int32)[None]
    assert np.allclose(O.sparse_attend(q, Kr, Vr, idx, 0.5), O.sparse_attend(q2, Kr, Vr, idx, 0.5), rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- synthetic workload, soft checks
def test_synthetic_layer_has_about_31_active_channels_at_B48():
    from workloads.synth import make_layer
    L = make_layer(4096, Hkv=8, Hq=32, seed=0)
    dep = O.alloc_depth(L.q.numpy(), L.var.numpy(), "waterfill", 48, 4)
    active = (dep > 0).sum(1)
    assert np.all(dep.sum(1) == 48)
    assert 24 <= active.mean() <= 38                          # the paper reports 30-34 on its models
    bits = np.mean([O.bits_per_token(r) for r in dep])
    assert 52 <= bits <= 59                                   # the paper's 56-bit read


def test_needles_are_selected_at_B48():
    from workloads.synth import make_layer
    L = make_layer(4096, Hkv=1, Hq=1, seed=0)
    K = L.K.numpy()
    planes, scales = O.build_planes(K)
    dep = O.alloc_depth(L.q.numpy(), L.var.numpy(), "waterfill", 48, 1)
    s = O.scan(planes, scales, L.q.numpy(), dep, 4096, 1)
    idx = O.topk(s, 64)
    assert set(L.needles[0].tolist()) <= set(idx[0].tolist())


# ---------------------------------------------------------------- O6 union of winners
def test_union_of_winners_properties():
    r = np.random.default_rng(9)
    Hkv, G, n, k, d = 3, 4, 500, 60, 8
    Kr = r.standard_normal((Hkv, n, d)).astype(np.float32)
    Vr = r.standard_normal((Hkv, n, d)).astype(np.float32)
    q = r.standard_normal((Hkv * G, d)).astype(np.float32)
    idx = np.stack([np.sort(r.permutation(n)[:k]) for _ in range(Hkv * G)]).astype(np.int32)
    idx[1] = idx[0]                                           # two heads with identical picks
    ul, Ks, Vs, loc = O.gather_union(idx, G, Kr, Vr)
    for kv in range(Hkv):
        u = ul[kv]
        assert np.all(np.diff(u) > 0) and k <= len(u) <= G * k             # ascending, distinct, bounded
        assert np.array_equal(u, np.unique(idx[kv * G:(kv + 1) * G]))       # library routine on the definition
        for h in range(kv * G, (kv + 1) * G):
            assert np.array_equal(u[loc[h]], idx[h])                        # positions map back to the picks
        assert np.array_equal(Ks[kv], Kr[kv][u]) and np.array_equal(Vs[kv], Vr[kv][u])
    assert len(ul[0]) <= 3 * k                                              # the duplicate head adds nothing
    # attention over the staged rows with the local indices is the attention over the original rows
    a = O.sparse_attend(q, Kr, Vr, idx, 0.3)
    cap = max(len(u) for u in ul)
    Kst = np.zeros((Hkv, cap, d), np.float32); Vst = np.zeros((Hkv, cap, d), np.float32)
    for kv in range(Hkv):
        Kst[kv, :len(ul[kv])] = Ks[kv]; Vst[kv, :len(ul[kv])] = Vs[kv]
    b = O.sparse_attend(q, Kst, Vst, loc, 0.3)
    assert np.array_equal(a, b)


# ---------------------------------------------------------------- O7 KLT-rotated store
def test_klt_rotation_properties():
    r = np.random.default_rng(12)
    Hkv, G, n, d = 2, 2, 400, 16
    A = r.standard_normal((Hkv, d, d))
    K = (r.standard_normal((Hkv, n, d)) @ A + r.standard_normal((Hkv, 1, d)) * 3).astype(np.float32)
    q = r.standard_normal((Hkv * G, d)).astype(np.float32)
    mu, C = O.calibrate(K)
    for h in range(Hkv):                                                    # library routines on the definitions
        assert np.allclose(mu[h], K[h].astype(np.float64).mean(0), rtol=0, atol=1e-12)
        assert np.allclose(C[h], np.cov(K[h].astype(np.float64), rowvar=False, ddof=1), rtol=1e-10, atol=1e-12)
    V, lam = O.klt_basis(C)
    Kr = O.rotate_keys(K, mu, V)
    qr = O.rotate_query(q, V, G)
    for h in range(Hkv):
        assert np.allclose(V[h].T @ V[h], np.eye(d), atol=1e-10)             # orthonormal basis
        assert np.all(np.diff(lam[h]) <= 1e-12)                              # largest variance first
        cov_rot = np.cov(Kr[h], rowvar=False, ddof=1)
        assert np.allclose(cov_rot, np.diag(lam[h]), atol=1e-8 * lam[h].max())   # rotated channels are uncorrelated,
        assert np.allclose(Kr[h].mean(0), 0, atol=1e-10)                     # centred, with variances lambda
    # scores are preserved up to a per-head constant: q.k = (qV).((k - mu)V) + q.mu
    for hq in range(Hkv * G):
        h = hq // G
        exact = K[h].astype(np.float64) @ q[hq].astype(np.float64)
        rot = Kr[h] @ qr[hq] + q[hq].astype(np.float64) @ mu[h]
        assert np.allclose(exact, rot, rtol=1e-10, atol=1e-9)
    # so the ranking, and with it the exact top-k set, is the same in both bases
    assert np.array_equal(O.topk(O.exact_scores(q, K), 20), O.topk(np.stack([Kr[h // G] @ qr[h] for h in range(Hkv * G)]), 20))


# ---------------------------------------------------------------- O8 per-channel statistics
def test_channel_variance_matches_the_worked_example_closed_forms_and_the_covariance_diagonal():
    import json, os
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "appendix_a_worked_example.json")))
    K = np.asarray(g["K"], dtype=np.float32)[None]                           # six keys, four channels
    _, var = O.channel_variance(K)
    assert np.allclose(var[0], g["var_printed"], atol=6e-4)                  # Appendix A prints n - 1 variances to 3 decimals
    # closed form: the integers 0 .. n-1 have mean (n - 1)/2 and unbiased variance n (n + 1) / 12
    n = 1000
    ramp = np.arange(n, dtype=np.float32)[None, :, None] * np.ones((1, 1, 3), np.float32)
    ramp[0, :, 1] += 5.0                                                      # a shift moves the mean only
    ramp[0, :, 2] *= -2.0                                                     # a scale multiplies the variance by its square
    mean, var = O.channel_variance(ramp)
    assert np.allclose(mean[0], [(n - 1) / 2, (n - 1) / 2 + 5, -(n - 1)], rtol=1e-13)
    assert np.allclose(var[0], [n * (n + 1) / 12, n * (n + 1) / 12, 4 * n * (n + 1) / 12], rtol=1e-13)
    # library routine and the diagonal of the session covariance (a different code path)
    K = rng_keys(3, 2, 777, 9)
    mean, var = O.channel_variance(K)
    mu, C = O.calibrate(K)
    for h in range(2):
        assert np.allclose(var[h], np.var(K[h].astype(np.float64), axis=0, ddof=1), rtol=1e-12)
        assert np.allclose(var[h], np.diag(C[h]), rtol=1e-12)
        assert np.allclose(mean[h], mu[h], rtol=0, atol=1e-13)
    # a single key has no spread
    _, v1 = O.channel_variance(K[:, :1])
    assert np.all(v1 == 0)


# ---------------------------------------------------------------- O9 per-layer budgets
def test_layer_budget_plan_hand_example():
    levels = [24, 32, 40, 48]
    #            24    32    40    48
    err = [[1.00, 0.50, 0.40, 0.39],     # layer 0: big first drop
           [1.00, 0.90, 0.30, 0.29],     # layer 1: the drop comes late
           [0.20, 0.19, 0.18, 0.17]]     # layer 2: flat
    # mean 32 -> 24 bits to hand out in steps of 8: layer 0 (0.50/8); then layers 0 and 1 both offer 0.10/8 and the
    # tie goes to layer 0; then layer 1 (0.10/8 against layer 0's 0.01/8)
    assert list(O.plan_layer_budgets(err, levels, 32)) == [2, 1, 0]
    # mean 40 -> 48 bits = 6 steps: continue 1 (0.60/8), then 0 (0.01/8) == 1 (0.01/8) == 2 (0.01/8) -> lower layer 0, then 1
    assert list(O.plan_layer_budgets(err, levels, 40)) == [3, 3, 0]
    # the floor and the ceiling
    assert list(O.plan_layer_budgets(err, levels, 24)) == [0, 0, 0]
    assert list(O.plan_layer_budgets(err, levels, 48)) == [3, 3, 3]
    assert list(O.plan_layer_budgets(err, levels, 1000)) == [3, 3, 3]
    # a target between two sums is never exceeded: mean 30 allows 18 extra bits = two steps
    assert list(O.plan_layer_budgets(err, levels, 30)) == [2, 0, 0]


@pytest.mark.parametrize("seed", range(6))
def test_layer_budget_plan_is_optimal_for_convex_error_curves(seed):
    """Marginal analysis: with evenly spaced levels and error curves that fall with diminishing returns, moving bits
    one level at a time to the steepest layer minimises the summed error among all plans of the same total."""
    r = np.random.default_rng(seed)
    L, nlev = 4, 5
    levels = [24 + 8 * i for i in range(nlev)]
    drops = -np.sort(-r.uniform(0.01, 1.0, size=(L, nlev - 1)), axis=1)       # decreasing drops = convex curve
    err = np.concatenate([np.full((L, 1), 5.0), 5.0 - np.cumsum(drops, axis=1)], axis=1)
    for steps in range(0, L * (nlev - 1) + 1, 3):
        target = (L * levels[0] + 8 * steps) / L
        plan = O.plan_layer_budgets(err, levels, target)
        assert plan.sum() == steps
        best = min(sum(err[l, c[l]] for l in range(L))
                   for c in itertools.product(range(nlev), repeat=L) if sum(c) == steps)
        assert abs(sum(err[l, plan[l]] for l in range(L)) - best) < 1e-12

"""CPU oracle for the Fathom decode-step hot path (TEST INFRASTRUCTURE ONLY).

This module is the slow, plain restatement of what the five calls of the
library compute (and of the calibration-time steps around them), written from the paper's definitions in numpy / fp64.  It is
imported only by the tests, by the smoke check and by the benchmark's
`cpu_baseline` / `--impl reference` legs.  It shares no code with the CUDA
path and never imports the product package; the product never imports it.

Every function cites the passage it follows.  Shapes:

    K        [Hkv][n][d]   float32   token-major keys
    planes   [Hkv][d][4][nb] uint64  nb = ceil(n/64); plane 0 = MSB (sign)
    scales   [Hkv][d][nb]  float16   stored cell width s = a/8
    q        [Hq][d]       float32   Hq = Hkv * G, head h belongs to KV head h // G
    var      [Hkv][d]      float32   per-channel key variance (an input)
    depth    [P][d]        uint8     P = Hq / heads_per_plan plans
    scores   [Hq][n]       float64
    idx      [Hq][k]       int32     ascending token indices

Parity status: every function below is pinned by tests/test_oracle_*.py to the
paper's worked example (Appendix A), to closed forms, or to brute force on
tiny inputs.  Nothing here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

BLOCK = 64          # tokens per scale block (Sec. 3.2)
NPLANES = 4         # bits per code (Sec. 3.2)


# --------------------------------------------------------------------------
# O1  plane builder  (Sec. 3.2, Eq. 2 and the paragraph after it)
# --------------------------------------------------------------------------
def quantise_block_codes(K: np.ndarray):
    """4-bit symmetric per-channel block codes (Eq. 2).

    For block beta (64 consecutive tokens; the tail block holds the real
    tokens only) and channel j:  a = max |k|,  the stored scale is
    S = fp16(a / 8) and the code is clip(floor(k / S), -8, 7) + 8.  The code is
    taken with the *stored* (fp16-rounded) scale: only this reading reproduces
    the approximate scores printed in Appendix A.  S == 0 gives code 8 (zero).

    Returns codes [Hkv][n][d] uint8 and scales [Hkv][d][nb] float16.
    """
    K = np.asarray(K, dtype=np.float32)
    Hkv, n, d = K.shape
    nb = (n + BLOCK - 1) // BLOCK
    codes = np.empty((Hkv, n, d), dtype=np.uint8)
    scales = np.zeros((Hkv, d, nb), dtype=np.float16)
    pad = nb * BLOCK - n
    for h in range(Hkv):
        # zero rows appended to the tail block do not change its max |k|; their codes are dropped
        blk = np.pad(K[h], ((0, pad), (0, 0))).reshape(nb, BLOCK, d)   # [nb][64][d] fp32
        a = np.max(np.abs(blk), axis=1)                         # [nb][d] fp32, exact
        with np.errstate(over="ignore"):
            S = (a / np.float32(8)).astype(np.float16)          # a/8 exact, then RN-even to fp16
        scales[h] = S.T
        s = S.astype(np.float64)[:, None, :]
        with np.errstate(divide="ignore", invalid="ignore"):
            # double division of an fp32 by an fp16 value: the real quotient of a
            # 24-bit by an 11-bit significand is either an integer or at least
            # 2^-24 (relative) away from one, so floor() of the fp64 quotient is
            # the floor of the real quotient.
            cell = np.floor(blk.astype(np.float64) / s)
        cell = np.where(s == 0.0, 0.0, cell)
        codes[h] = (np.clip(cell, -8, 7) + 8).astype(np.uint8).reshape(nb * BLOCK, d)[:n]
    return codes, scales


def pack_planes(codes: np.ndarray) -> np.ndarray:
    """Channel-major bit planes (Sec. 3.2, paragraph after Eq. 2).

    Bit p (0 = most significant) of the 64 codes of (block, channel) becomes one
    64-bit word; token i sits at bit (i mod 64), lowest token = least significant
    bit; absent tail tokens contribute 0 bits.
    """
    Hkv, n, d = codes.shape
    nb = (n + BLOCK - 1) // BLOCK
    planes = np.zeros((Hkv, d, NPLANES, nb), dtype=np.uint64)
    for i in range(n):
        b, r = divmod(i, BLOCK)
        c = codes[:, i, :].astype(np.uint64)                    # [Hkv][d]
        for p in range(NPLANES):
            bit = (c >> np.uint64(3 - p)) & np.uint64(1)
            planes[:, :, p, b] |= bit << np.uint64(r)
    return planes


def pack_planes_fast(codes: np.ndarray) -> np.ndarray:
    """Same result as pack_planes, vectorised with numpy bit packing (used for large n;
    a test checks it word for word against the loop version)."""
    Hkv, n, d = codes.shape
    nb = (n + BLOCK - 1) // BLOCK
    pad = nb * BLOCK - n
    c = np.pad(codes, ((0, 0), (0, pad), (0, 0)))               # absent tokens -> bits 0
    planes = np.empty((Hkv, d, NPLANES, nb), dtype=np.uint64)
    for p in range(NPLANES):
        bit = ((c >> (3 - p)) & 1).astype(np.uint8)             # [Hkv][nb*64][d]
        bit = np.ascontiguousarray(bit.transpose(0, 2, 1))      # [Hkv][d][nb*64]
        by = np.packbits(bit, axis=-1, bitorder="little")       # [Hkv][d][nb*8] bytes
        planes[:, :, p, :] = by.reshape(Hkv, d, nb, 8).copy().view("<u8").reshape(Hkv, d, nb)
    return planes


def build_planes(K: np.ndarray):
    """O1: K -> (planes, scales).  Sec. 3.2."""
    codes, scales = quantise_block_codes(K)
    return pack_planes_fast(codes), scales


def unpack_codes(planes: np.ndarray, n: int, t: int = NPLANES) -> np.ndarray:
    """Reads the first t planes and returns c^(t) = c >> (4 - t) per token
    (Sec. 3.2: a prefix of t planes is the t-bit code).  [Hkv][d][n] uint8."""
    Hkv, d, _, nb = planes.shape
    out = np.zeros((Hkv, d, nb * BLOCK), dtype=np.uint8)
    for p in range(t):
        by = np.ascontiguousarray(planes[:, :, p, :]).astype("<u8").view(np.uint8)
        bits = np.unpackbits(by.reshape(Hkv, d, nb * 8), axis=-1, bitorder="little")
        out = (out << 1) | bits
    return out[:, :, :n]


# --------------------------------------------------------------------------
# O2  depth allocation  (Sec. 3.3, Eq. 3 and Eq. 4; Appendix A)
# --------------------------------------------------------------------------
def importance(q: np.ndarray, var: np.ndarray, heads_per_plan: int) -> np.ndarray:
    """g_j = sum_h (q_j^(h))^2 * Var(k_j)  (Eq. 3), summed over the heads of a plan
    in ascending head order, in fp64.  Returns [P][d]."""
    q = np.asarray(q, dtype=np.float32).astype(np.float64)
    var = np.asarray(var, dtype=np.float32).astype(np.float64)
    Hq, d = q.shape
    Hkv = var.shape[0]
    G = Hq // Hkv
    P = Hq // heads_per_plan
    g = np.zeros((P, d), dtype=np.float64)
    for pl in range(P):
        acc = np.zeros(d, dtype=np.float64)
        for h in range(pl * heads_per_plan, (pl + 1) * heads_per_plan):
            acc = acc + q[h] * q[h]
        g[pl] = acc * var[(pl * heads_per_plan) // G]
    return g


def waterfill_depths(g: np.ndarray, B: int) -> np.ndarray:
    """Integer reverse water-filling (Eq. 4) for one plan, in exact form.

    round(log4(g_j / theta)) >= m  <=>  theta <= 2 * g_j * 4^-m, so at water line
    theta channel j holds every plane m in 1..4 whose priority pi = g_j 4^-m satisfies
    2 pi >= theta.  The water line of Sec. 3.3 (the least theta whose depths still fit B)
    therefore admits the longest prefix (at most B items) of the planes sorted by priority.  Ties: lower channel,
    then lower plane.  Zero priorities sort last, so B >= 4d gives depth 4 everywhere.
    """
    g = np.asarray(g, dtype=np.float64)
    d = g.shape[0]
    items = []
    for j in range(d):
        for m in range(1, NPLANES + 1):
            items.append((-(g[j] * 4.0 ** (-m)), j, m))         # 4^-m scaling is exact
    items.sort()
    t = np.zeros(d, dtype=np.uint8)
    for _, j, _m in items[:max(0, min(int(B), NPLANES * d))]:
        t[j] += 1
    return t


def depths_at_theta(g: np.ndarray, theta: float) -> np.ndarray:
    """Eq. 4 evaluated literally at one water line (round = half away from zero; g = 0
    gives depth 0)."""
    g = np.asarray(g, dtype=np.float64)
    with np.errstate(divide="ignore"):
        x = np.log(g / theta) / np.log(4.0)
    x = np.where(g > 0, x, -np.inf)
    r = np.where(np.isfinite(x), np.floor(x + 0.5), -1e9)
    return np.clip(r, 0, NPLANES).astype(np.uint8)


def waterfill_depths_bisection(g: np.ndarray, B: int, lo: float, hi: float, steps: int = 30):
    """The paper's literal search (Sec. 3.3, Appendix A): `steps` bisections on
    log(theta); a trial whose depths overflow B becomes the lower end, otherwise the
    upper end; the answer is the depths at the upper end.  Returns (depths, theta_hi,
    trace) where trace lists (lo, hi, trial, depths, sum) per step."""
    trace = []
    for _ in range(steps):
        mid = float(np.sqrt(lo * hi))
        t = depths_at_theta(g, mid)
        s = int(t.sum())
        trace.append((lo, hi, mid, t.copy(), s))
        if s > B:
            lo = mid
        else:
            hi = mid
    return depths_at_theta(g, hi), hi, trace


def fixed_channel_depths(q: np.ndarray, heads_per_plan: int, r: int) -> np.ndarray:
    """Fixed-channel mode (SparQ's grouped-query rule, Sec. 2 and Appendix A): the r
    channels with the largest sum_h |q_j^(h)| are read at depth 4, the rest at 0; ties
    go to the lower channel.  Returns [P][d]."""
    q = np.asarray(q, dtype=np.float32).astype(np.float64)
    Hq, d = q.shape
    P = Hq // heads_per_plan
    out = np.zeros((P, d), dtype=np.uint8)
    for pl in range(P):
        w = np.zeros(d, dtype=np.float64)
        for h in range(pl * heads_per_plan, (pl + 1) * heads_per_plan):
            w = w + np.abs(q[h])
        order = sorted(range(d), key=lambda j: (-w[j], j))
        for j in order[:max(0, min(int(r), d))]:
            out[pl, j] = NPLANES
    return out


def alloc_depth(q, var, mode: str, budget: int, heads_per_plan: int) -> np.ndarray:
    """O2: depth plans [P][d].  mode in {"waterfill", "fixed_top_r", "uniform"}."""
    q = np.asarray(q, dtype=np.float32)
    Hq, d = q.shape
    P = Hq // heads_per_plan
    if mode == "waterfill":
        g = importance(q, var, heads_per_plan)
        return np.stack([waterfill_depths(g[pl], budget) for pl in range(P)])
    if mode == "fixed_top_r":
        return fixed_channel_depths(q, heads_per_plan, budget)
    if mode == "uniform":
        return np.full((P, d), min(max(int(budget), 0), NPLANES), dtype=np.uint8)
    raise ValueError(mode)


# --------------------------------------------------------------------------
# O3  scan  (Sec. 3.2 prefix dequantiser; Sec. 3.3: a channel of depth 0 is not read and adds nothing)
# --------------------------------------------------------------------------
def prefix_values(planes, scales, n: int, h: int, j: int, t: int) -> np.ndarray:
    """Dequantised value of channel j of KV head h for every token, read to depth t:
    (c^(t) + 1/2 - 2^(t-1)) * a / 2^(t-1) with a = 8 * S of the token's block (Sec. 3.2)."""
    c = unpack_codes(planes[h:h + 1, j:j + 1], n, t)[0, 0].astype(np.float64)
    a = 8.0 * np.repeat(scales[h, j].astype(np.float64), BLOCK)[:n]
    return (c + 0.5 - 2.0 ** (t - 1)) * a / 2.0 ** (t - 1)


def scan(planes, scales, q, depth, n: int, heads_per_plan: int) -> np.ndarray:
    """O3: approximate scores  s_i^(h) = sum_{j: t_j>0} q_j^(h) * khat_ij^(t_j), channels in
    ascending order, fp64, no 1/sqrt(d) factor (Appendix A prints unscaled scores)."""
    q = np.asarray(q, dtype=np.float32).astype(np.float64)
    Hq, d = q.shape
    Hkv = planes.shape[0]
    G = Hq // Hkv
    scores = np.zeros((Hq, n), dtype=np.float64)
    for pl in range(Hq // heads_per_plan):
        kv = (pl * heads_per_plan) // G
        for j in range(d):
            t = int(depth[pl, j])
            if t == 0:
                continue
            v = prefix_values(planes, scales, n, kv, j, t)
            for h in range(pl * heads_per_plan, (pl + 1) * heads_per_plan):
                scores[h] += q[h, j] * v
    return scores


def scan_signed_planes(planes, scales, q, depth, n: int, heads_per_plan: int) -> np.ndarray:
    """Independent second formulation of O3 used as a cross-check: a t-plane read is
    a * sum_{p<t} (2 bit_p - 1) 2^-(p+1)."""
    q = np.asarray(q, dtype=np.float32).astype(np.float64)
    Hq, d = q.shape
    Hkv, _, _, nb = planes.shape
    G = Hq // Hkv
    scores = np.zeros((Hq, n), dtype=np.float64)
    for pl in range(Hq // heads_per_plan):
        kv = (pl * heads_per_plan) // G
        for j in range(d):
            a = 8.0 * np.repeat(scales[kv, j].astype(np.float64), BLOCK)[:n]
            v = np.zeros(n, dtype=np.float64)
            for p in range(int(depth[pl, j])):
                by = np.ascontiguousarray(planes[kv, j, p]).astype("<u8").view(np.uint8)
                bit = np.unpackbits(by, bitorder="little")[:n].astype(np.float64)
                v += (2.0 * bit - 1.0) * 2.0 ** (-(p + 1))
            for h in range(pl * heads_per_plan, (pl + 1) * heads_per_plan):
                scores[h] += q[h, j] * (a * v)
    return scores


def scan_tokens(planes, scales, q, depth, heads_per_plan: int, h: int, tokens) -> np.ndarray:
    """O3 for one query head at a few sampled token indices (used to spot-check
    full-size runs one output at a time).  Same formula and channel order as scan()."""
    q = np.asarray(q, dtype=np.float32).astype(np.float64)
    Hq, d = q.shape
    Hkv = planes.shape[0]
    G = Hq // Hkv
    pl, kv = h // heads_per_plan, h // G
    out = np.zeros(len(tokens), dtype=np.float64)
    for n_i, i in enumerate(tokens):
        b, r = divmod(int(i), BLOCK)
        s = 0.0
        for j in range(d):
            t = int(depth[pl, j])
            if t == 0:
                continue
            c = 0
            for p in range(t):
                c = (c << 1) | ((int(planes[kv, j, p, b]) >> r) & 1)
            a = 8.0 * float(scales[kv, j, b])
            s += q[h, j] * ((c + 0.5 - 2.0 ** (t - 1)) * a / 2.0 ** (t - 1))
        out[n_i] = s
    return out


def bits_per_token(depth_row: np.ndarray) -> float:
    """Byte-accounting convention (Sec. 4): code bits read plus 16 bits per 64 tokens for
    the fp16 scale of every channel read, i.e. B + A/4."""
    t = np.asarray(depth_row).astype(np.int64)
    return float(t.sum()) + float((t > 0).sum()) * 16.0 / BLOCK


# --------------------------------------------------------------------------
# O4  top-k  (Sec. 2 "Top-k decoding": sink + local always kept, the rest by score)
# --------------------------------------------------------------------------
def topk(scores: np.ndarray, k: int, n_sink: int = 0, n_local: int = 0) -> np.ndarray:
    """O4: per query head, forced set F = first n_sink and last n_local tokens; the
    remaining k - |F| are the highest scores among the other tokens, ties to the lower
    index (a full stable sort); -0 equals +0.  Returns ascending indices [Hq][k] int32."""
    scores = np.asarray(scores)
    Hq, n = scores.shape
    out = np.empty((Hq, k), dtype=np.int32)
    forced = np.zeros(n, dtype=bool)
    forced[:min(n_sink, n)] = True
    if n_local > 0:
        forced[max(0, n - n_local):] = True
    nf = int(forced.sum())
    assert nf <= k <= n
    free = np.nonzero(~forced)[0]
    for h in range(Hq):
        s = scores[h, free] + 0.0                               # -0 + 0 = +0
        order = np.argsort(-s, kind="stable")                   # stable: equal keys keep index order
        win = free[order[:k - nf]]
        out[h] = np.sort(np.concatenate([np.nonzero(forced)[0], win])).astype(np.int32)
    return out


# --------------------------------------------------------------------------
# O5  exact attention over the selected rows  (Sec. 2 "Top-k decoding")
# --------------------------------------------------------------------------
def sparse_attend(q, Krows, Vrows, idx, softmax_scale: float) -> np.ndarray:
    """O5: o = softmax(scale * q K_S^T) V_S per query head over its own index list;
    rows are used at their stored precision widened to fp64.  Returns [Hq][d] fp64."""
    q = np.asarray(q, dtype=np.float32).astype(np.float64)
    Hq, d = q.shape
    Hkv = Krows.shape[0]
    G = Hq // Hkv
    out = np.zeros((Hq, d), dtype=np.float64)
    for h in range(Hq):
        kv = h // G
        S = np.asarray(idx[h], dtype=np.int64)
        Ks = np.asarray(Krows[kv][S], dtype=np.float64)
        Vs = np.asarray(Vrows[kv][S], dtype=np.float64)
        e = (Ks @ q[h]) * float(softmax_scale)
        e = e - e.max()
        w = np.exp(e)
        out[h] = (w / w.sum()) @ Vs
    return out


def dense_attention(q, Krows, Vrows, softmax_scale: float) -> np.ndarray:
    """Dense softmax attention over all n rows (the error reference of Sec. 4 "Fidelity metric")."""
    n = Krows.shape[1]
    Hq = np.asarray(q).shape[0]
    idx = np.broadcast_to(np.arange(n, dtype=np.int32), (Hq, n))
    return sparse_attend(q, Krows, Vrows, idx, softmax_scale)


def exact_scores(q, Krows) -> np.ndarray:
    """Unscaled exact scores q . k per query head (Appendix A "exact scores")."""
    q = np.asarray(q, dtype=np.float32).astype(np.float64)
    Hq, d = q.shape
    Hkv = Krows.shape[0]
    G = Hq // Hkv
    return np.stack([np.asarray(Krows[h // G], dtype=np.float64) @ q[h] for h in range(Hq)])


# --------------------------------------------------------------------------
# O6  union of a group's winners  (Sec. 1: the union of the G heads' winners is fetched once per KV head;
#     Sec. 4 "Offload harness": the row fetch of a step is that union)
# --------------------------------------------------------------------------
def gather_union(idx: np.ndarray, G: int, Krows, Vrows):
    """O6: per KV head kv, the ascending list u of distinct tokens picked by its G query heads, the rows
    K[kv][u], V[kv][u], and every pick rewritten as its position in u.
    Returns (ulists [list of arrays], K_stage [list], V_stage [list], idx_local [Hq][k] int32)."""
    idx = np.asarray(idx)
    Hq, k = idx.shape
    Hkv = Hq // G
    ulists, Ks, Vs = [], [], []
    idx_local = np.empty((Hq, k), dtype=np.int32)
    for kv in range(Hkv):
        picks = set()
        for h in range(kv * G, (kv + 1) * G):
            picks |= set(int(t) for t in idx[h])
        u = np.array(sorted(picks), dtype=np.int64)
        pos = {int(t): p for p, t in enumerate(u)}
        for h in range(kv * G, (kv + 1) * G):
            idx_local[h] = [pos[int(t)] for t in idx[h]]
        ulists.append(u)
        Ks.append(np.asarray(Krows[kv])[u])
        Vs.append(np.asarray(Vrows[kv])[u])
    return ulists, Ks, Vs, idx_local


# --------------------------------------------------------------------------
# O7  KLT-rotated store  (Sec. 3.5 "Basis rule"; Appendix B5 session calibration)
# --------------------------------------------------------------------------
def calibrate(K: np.ndarray):
    """Per KV head: mean mu[d] and covariance C[d][d] of the session's own keys (Appendix B5: the statistics of the
    calibration-free variant are taken from the keys the session itself has cached, head by head); unbiased (n - 1),
    fp64.  Returns (mu [Hkv][d], C [Hkv][d][d])."""
    K = np.asarray(K, dtype=np.float32).astype(np.float64)
    Hkv, n, d = K.shape
    mu = K.mean(axis=1)
    C = np.empty((Hkv, d, d))
    for h in range(Hkv):
        X = K[h] - mu[h]
        C[h] = X.T @ X / max(n - 1, 1)
    return mu, C


def klt_basis(C: np.ndarray):
    """Eigenbasis V (columns = directions) and eigenvalues lambda of each covariance, largest variance first.
    (The order of the directions does not change what is read: the depth rule ranks them by g_j anyway.)"""
    Hkv, d, _ = C.shape
    V = np.empty((Hkv, d, d))
    lam = np.empty((Hkv, d))
    for h in range(Hkv):
        w, U = np.linalg.eigh(C[h])
        order = np.argsort(-w, kind="stable")
        lam[h] = np.maximum(w[order], 0.0)
        V[h] = U[:, order]
    return V, lam


def rotate_keys(K: np.ndarray, mu: np.ndarray, V: np.ndarray) -> np.ndarray:
    """(k - mu) V per KV head (Sec. 3.5: the rotated keys whose planes the store keeps), fp64."""
    K = np.asarray(K, dtype=np.float32).astype(np.float64)
    return np.stack([(K[h] - np.asarray(mu, dtype=np.float64)[h]) @ np.asarray(V, dtype=np.float64)[h] for h in range(K.shape[0])])


def rotate_query(q: np.ndarray, V: np.ndarray, G: int) -> np.ndarray:
    """q^(h) V of the head's KV head (Sec. 3.5: g_j = sum_h ((q^(h) V)_j)^2 lambda_j), fp64."""
    q = np.asarray(q, dtype=np.float32).astype(np.float64)
    return np.stack([q[h] @ np.asarray(V, dtype=np.float64)[h // G] for h in range(q.shape[0])])


# --------------------------------------------------------------------------
# O8  per-channel key statistics  (Sec. 3.3: Var(k_j) in the importance g_j; Appendix B5: taken from the
#     session's own keys)
# --------------------------------------------------------------------------
def channel_variance(K: np.ndarray):
    """Per (KV head, channel): mean and unbiased sample variance  sum_i (k_ij - mean_j)^2 / (n - 1)  of the
    session's keys, written out as the definition in fp64 (Appendix A prints n - 1 values).
    Returns (mean [Hkv][d], var [Hkv][d])."""
    K = np.asarray(K, dtype=np.float32).astype(np.float64)
    Hkv, n, d = K.shape
    mean = np.empty((Hkv, d))
    var = np.empty((Hkv, d))
    for h in range(Hkv):
        for j in range(d):
            col = K[h, :, j]
            m = col.sum() / n
            mean[h, j] = m
            dev = col - m
            var[h, j] = (dev * dev).sum() / max(n - 1, 1)
    return mean, var


# --------------------------------------------------------------------------
# O9  per-layer budgets  (Sec. 3.4 "Per-layer budgets")
# --------------------------------------------------------------------------
def plan_layer_budgets(err: np.ndarray, levels, target_mean: float) -> np.ndarray:
    """Greedy per-layer plan: budgets B_l from the ascending list `levels` (the paper's range is 24..128) at a
    target mean.  err[l][i] is the measured error of layer l at budget levels[i].  Every layer starts at the
    lowest level; each step raises one layer by one level, namely the layer with the largest error drop per added
    bit  (err[l][i] - err[l][i+1]) / (levels[i+1] - levels[i]),  ties to the lower layer; a step is admissible
    while the sum of budgets stays <= target_mean * L; the plan is final when no step is admissible.
    (The paper fixes neither the start nor the step; this reading moves bits one level at a time from the floor.)
    Returns the level INDEX per layer."""
    err = np.asarray(err, dtype=np.float64)
    levels = [int(b) for b in levels]
    L, nlev = err.shape
    assert nlev == len(levels) and all(levels[i] < levels[i + 1] for i in range(nlev - 1))
    cur = np.zeros(L, dtype=np.int64)
    total = L * levels[0]
    cap = float(target_mean) * L
    while True:
        best, best_gain = -1, 0.0
        for l in range(L):
            i = int(cur[l])
            if i + 1 >= nlev:
                continue
            step = levels[i + 1] - levels[i]
            if total + step > cap:
                continue
            gain = (err[l, i] - err[l, i + 1]) / step
            if best < 0 or gain > best_gain:
                best, best_gain = l, gain
        if best < 0:
            return cur
        total += levels[int(cur[best]) + 1] - levels[int(cur[best])]
        cur[best] += 1

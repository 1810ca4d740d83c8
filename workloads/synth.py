"""Seeded synthetic decode-step inputs (shared by the CUDA path's tests/bench and by the oracle's tests).

This module only draws random inputs; it contains none of the method's arithmetic
(no quantiser, no depth rule, no scan, no selection, no attention).  The recipe
stands in for one layer of a Qwen3-8B-shaped KV cache (Sec. 1: 8 KV heads of 128
channels, 4 query heads per KV head):

* per channel a standard deviation sigma_c = exp(U[ln 0.1, ln 4]); 4 distinct outlier
  channels per KV head at sigma = 16;  K[i][c] ~ N(0, sigma_c^2) in fp32;
* q[h] ~ N(0, 1)^d in fp32 per query head;
* 8 needle tokens per KV head (two per query head of a 4-head group; all 8 for a
  single-head problem) at distinct positions in [64, n-64): the key there is
  rho * (0.9 qhat + sqrt(1 - 0.81) zhat), zhat a unit Gaussian direction made
  orthogonal to qhat, rho = sqrt(sum_c sigma_c^2) (a typical key norm), so cos(k, q) = 0.9;
* V ~ N(0,1) rounded to bf16; the rows used by exact attention are bf16(K);
* var = unbiased sample variance of K over tokens per (KV head, channel), computed in
  fp64 and rounded to fp32 (the session-calibrated statistic of Appendix B5; an INPUT
  of the depth allocator, so both sides consume the same array).

Everything is generated with one seeded torch.Generator on the requested device; the
caller copies tensors to the other side so both see identical bytes.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch


@dataclass
class LayerInputs:
    K: torch.Tensor        # [Hkv][n][d] float32
    Krows: torch.Tensor    # [Hkv][n][d] bfloat16  (= bf16(K))
    Vrows: torch.Tensor    # [Hkv][n][d] bfloat16
    q: torch.Tensor        # [Hq][d] float32
    var: torch.Tensor      # [Hkv][d] float32
    sigma: torch.Tensor    # [Hkv][d] float32
    needles: torch.Tensor  # [Hkv][8] int64 token positions
    n: int
    Hkv: int
    Hq: int
    d: int


def mix_seed(seed0: int, session: int = 0, layer: int = 0) -> int:
    """Deterministic 63-bit seed from (seed0, session, layer) (SplitMix64 finaliser)."""
    x = (seed0 * 0x9E3779B97F4A7C15 + session * 0xBF58476D1CE4E5B9 + layer * 0x94D049BB133111EB + 1) & (2**64 - 1)
    x ^= x >> 30
    x = (x * 0xBF58476D1CE4E5B9) & (2**64 - 1)
    x ^= x >> 27
    x = (x * 0x94D049BB133111EB) & (2**64 - 1)
    x ^= x >> 31
    return x & (2**63 - 1)


def make_layer(n: int, Hkv: int = 8, Hq: int = 32, d: int = 128, seed: int = 0,
               session: int = 0, layer: int = 0, device: str = "cpu",
               want_rows: bool = True, sigma_lo: float = 0.1, sigma_hi: float = 4.0, n_outliers: int = 4) -> LayerInputs:
    """sigma_lo, sigma_hi, n_outliers: the channel spread of the recipe (defaults: the recipe of the module docstring);
    the per-layer budget experiments vary them from layer to layer, as real layers differ in how concentrated they are."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(mix_seed(seed, session, layer))
    G = Hq // Hkv

    u = torch.rand(Hkv, d, generator=gen, device=dev, dtype=torch.float64)
    sigma = torch.exp(math.log(sigma_lo) + u * (math.log(sigma_hi) - math.log(sigma_lo)))
    for h in range(Hkv):
        out_ch = torch.randperm(d, generator=gen, device=dev)[:4]
        sigma[h, out_ch[:n_outliers]] = 16.0
    sigma = sigma.to(torch.float32)

    q = torch.randn(Hq, d, generator=gen, device=dev, dtype=torch.float32)

    K = torch.empty(Hkv, n, d, device=dev, dtype=torch.float32)
    for h in range(Hkv):            # per head keeps the transient small at n = 1M
        K[h] = torch.randn(n, d, generator=gen, device=dev, dtype=torch.float32) * sigma[h]

    # needles
    n_needles = 8
    needles = torch.zeros(Hkv, n_needles, dtype=torch.int64, device=dev)
    if n >= 128 + n_needles:
        for h in range(Hkv):
            pos = 64 + torch.randperm(n - 128, generator=gen, device=dev)[:n_needles]
            needles[h] = pos
            rho = torch.sqrt((sigma[h].double() ** 2).sum())
            for m in range(n_needles):
                qh = q[h * G + (m * G) // n_needles].double()      # two needles per head when G = 4
                qhat = qh / qh.norm()
                z = torch.randn(d, generator=gen, device=dev, dtype=torch.float64)
                z = z - (z @ qhat) * qhat
                zhat = z / z.norm()
                K[h, pos[m]] = (rho * (0.9 * qhat + math.sqrt(1.0 - 0.81) * zhat)).float()

    var = torch.stack([K[h].double().var(dim=0, unbiased=True) for h in range(Hkv)]).float() \
        if n > 1 else torch.ones(Hkv, d, device=dev)

    if want_rows:
        Krows = K.to(torch.bfloat16)
        Vrows = torch.empty(Hkv, n, d, device=dev, dtype=torch.bfloat16)
        for h in range(Hkv):
            Vrows[h] = torch.randn(n, d, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    else:
        Krows = Vrows = torch.empty(0, device=dev, dtype=torch.bfloat16)

    return LayerInputs(K=K, Krows=Krows, Vrows=Vrows, q=q, var=var, sigma=sigma,
                       needles=needles, n=n, Hkv=Hkv, Hq=Hq, d=d)


def session_lengths(n_sessions: int = 16, lo: int = 65536, hi: int = 1048576, seed: int = 0):
    """Context lengths of the multi-session batch: n_s = round(exp(U[ln lo, ln hi])), not
    forced to a multiple of 64."""
    gen = torch.Generator().manual_seed(mix_seed(seed, 10_000, 0))
    u = torch.rand(n_sessions, generator=gen, dtype=torch.float64)
    return [int(round(math.exp(math.log(lo) + float(x) * (math.log(hi) - math.log(lo))))) for x in u]

"""Seeded synthetic input generators shared by the tests, the benchmark and the oracle harness.

Nothing in this module performs any of the method's arithmetic (no encode, no Top-k, no
postings, no scoring): it only produces input tensors. Every value is a pure function of
(seed, tensor id, row, column) through a counter-based integer hash, so any row range of
any tensor can be regenerated on its own, on the CPU or on a CUDA device, with identical
bits (integer ops and a table lookup only; no device-side transcendental functions).

The distributions follow the five workload descriptions of the benchmark definition:
N(0,1) activations, per-channel lognormal scales with a few outlier channels, unit-norm
encoder columns, Gaussian biases, Gamma(2,1) lexical scores and a Zipf-skewed low-rank
mean shift.
"""
from __future__ import annotations

import math

import torch

_M32 = 0xFFFFFFFF
# Odd multipliers below 2**31 so that (32-bit value) * multiplier never overflows int64.
_C1 = 0x2C1B3C6D
_C2 = 0x297A2D39
_C3 = 0x1B873593
_GOLD = 0x1E3779B1

# tensor ids (the "stream" a value belongs to)
TID_X = 1
TID_W = 2
TID_BENC = 3
TID_BDEC = 4
TID_SCALE = 5
TID_OUTLIER = 6
TID_BM25_A = 7
TID_BM25_B = 8
TID_ZIPF_RANK = 9
TID_ZIPF_PI = 10
TID_QUERY_X = 11

_TABLE_BITS = 16
_table_cache: dict[str, torch.Tensor] = {}


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """Bijective 32-bit integer mixer evaluated in int64 (xorshift-multiply rounds)."""
    x = x & _M32
    x = (((x >> 16) ^ x) * _C1) & _M32
    x = (((x >> 15) ^ x) * _C2) & _M32
    x = (((x >> 13) ^ x) * _C3) & _M32
    x = (x >> 16) ^ x
    return x


def _mix32_int(v: int) -> int:
    v &= _M32
    v = (((v >> 16) ^ v) * _C1) & _M32
    v = (((v >> 15) ^ v) * _C2) & _M32
    v = (((v >> 13) ^ v) * _C3) & _M32
    return (v >> 16) ^ v


def hash_u32(seed: int, tid: int, rows: torch.Tensor, cols: torch.Tensor) -> torch.Tensor:
    """32-bit hash of (seed, tid, row, col) as an int64 tensor broadcast over rows x cols."""
    key = _mix32_int(seed * _GOLD + tid * 0x632BE5AB + 0x51ED27)
    h = _mix32(rows.to(torch.int64) ^ key)
    h = _mix32((h + cols.to(torch.int64) * _GOLD) & _M32)
    return h


def normal_table(device) -> torch.Tensor:
    """2**16 standard-normal quantiles (bin mid-points), computed once in fp64 on the host."""
    dev = str(device)
    if dev not in _table_cache:
        if "cpu" not in _table_cache:
            n = 1 << _TABLE_BITS
            p = (torch.arange(n, dtype=torch.float64) + 0.5) / n
            _table_cache["cpu"] = torch.special.ndtri(p).to(torch.float32)
        _table_cache[dev] = _table_cache["cpu"].to(device)
    return _table_cache[dev]


def normal(seed: int, tid: int, row0: int, n_rows: int, n_cols: int, device="cpu") -> torch.Tensor:
    """fp32 [n_rows, n_cols] of N(0,1) draws for rows row0 .. row0+n_rows-1 of tensor `tid`."""
    rows = torch.arange(row0, row0 + n_rows, dtype=torch.int64, device=device).unsqueeze(1)
    cols = torch.arange(n_cols, dtype=torch.int64, device=device).unsqueeze(0)
    h = hash_u32(seed, tid, rows, cols)
    return normal_table(device)[h >> (32 - _TABLE_BITS)]


def uniform01(seed: int, tid: int, row0: int, n_rows: int, n_cols: int) -> torch.Tensor:
    """fp64 uniforms in (0,1) on the host (24 hash bits, bin mid-points)."""
    rows = torch.arange(row0, row0 + n_rows, dtype=torch.int64).unsqueeze(1)
    cols = torch.arange(n_cols, dtype=torch.int64).unsqueeze(0)
    h = hash_u32(seed, tid, rows, cols)
    return ((h >> 8).to(torch.float64) + 0.5) / float(1 << 24)


def channel_scale(seed: int, d_in: int, sigma: float, outlier_frac: float, outlier_gain: float) -> torch.Tensor:
    """Per-channel scale exp(sigma * n_c) with ceil(outlier_frac * d_in) seeded channels multiplied
    by outlier_gain. Host fp32; sigma == 0 and outlier_frac == 0 gives all ones."""
    n = normal(seed, TID_SCALE, 0, 1, d_in)[0].to(torch.float64)
    s = torch.exp(sigma * n)
    n_out = int(math.ceil(outlier_frac * d_in)) if outlier_frac > 0 else 0
    if n_out:
        score = hash_u32(seed, TID_OUTLIER, torch.zeros(1, dtype=torch.int64), torch.arange(d_in))
        idx = torch.argsort(score, stable=True)[:n_out]
        s[idx] = s[idx] * outlier_gain
    return s.to(torch.float32)


def activations(seed: int, layer: int, row0: int, n_rows: int, d_in: int, dtype: torch.dtype,
                scale: torch.Tensor | None = None, device="cpu", tid: int = TID_X) -> torch.Tensor:
    """Key/query projection rows x[t, c] = scale[c] * g[t, c], g ~ N(0,1); one stream per layer."""
    g = normal(seed + 7919 * layer, tid, row0, n_rows, d_in, device)
    if scale is not None:
        g = g * scale.to(device)
    return g.to(dtype)


def sae_weights(seed: int, layer: int, d_in: int, d_sae: int, dtype: torch.dtype, device="cpu"):
    """Encoder parameters of one SAE: W_enc [d_in, d_sae] with unit-l2 columns (feature f = column f),
    b_enc ~ N(0, 0.1^2), b_dec ~ N(0, 0.05^2). Biases are fp32; W_enc has the activations' dtype."""
    s = seed + 104729 * layer
    w = normal(s, TID_W, 0, d_in, d_sae, device).to(torch.float64)
    w = w / torch.sqrt((w * w).sum(dim=0, keepdim=True))
    w = w.to(torch.float32).to(dtype).contiguous()
    b_enc = (0.1 * normal(s, TID_BENC, 0, 1, d_sae, device)[0]).contiguous()
    b_dec = (0.05 * normal(s, TID_BDEC, 0, 1, d_in, device)[0]).contiguous()
    return w, b_enc, b_dec


def gamma21(seed: int, n_rows: int, n_cols: int) -> torch.Tensor:
    """Host fp32 [n_rows, n_cols] of Gamma(shape 2, scale 1) draws: -ln(u1) - ln(u2)."""
    u1 = uniform01(seed, TID_BM25_A, 0, n_rows, n_cols)
    u2 = uniform01(seed, TID_BM25_B, 0, n_rows, n_cols)
    return (-(torch.log(u1) + torch.log(u2))).to(torch.float32)


def zipf_ranks(seed: int, layer: int, row0: int, n_rows: int, n_ranks: int, exponent: float, device="cpu"):
    """int64 [n_rows] ranks in [0, n_ranks) with P(r) proportional to (r+1)^-exponent; integer
    inverse-CDF lookup so host and device agree bit for bit."""
    w = torch.arange(1, n_ranks + 1, dtype=torch.float64) ** (-exponent)
    cdf = torch.cumsum(w / w.sum(), 0)
    thresh = torch.clamp((cdf * float(1 << 32)).round().to(torch.int64), max=(1 << 32) - 1)
    thresh[-1] = (1 << 32) - 1
    rows = torch.arange(row0, row0 + n_rows, dtype=torch.int64, device=device)
    h = hash_u32(seed + 7919 * layer, TID_ZIPF_RANK, rows, torch.zeros(1, dtype=torch.int64, device=device))
    return torch.searchsorted(thresh.to(device), h, right=False).clamp_(max=n_ranks - 1)


def zipf_popular_features(seed: int, layer: int, d_sae: int, n_ranks: int) -> torch.Tensor:
    """Seeded choice of n_ranks distinct 'popular' feature ids (host int64), rank order."""
    score = hash_u32(seed + 7919 * layer, TID_ZIPF_PI, torch.zeros(1, dtype=torch.int64), torch.arange(d_sae))
    return torch.argsort(score, stable=True)[:n_ranks]


def zipf_shifted_activations(seed: int, layer: int, row0: int, n_rows: int, w_enc: torch.Tensor,
                             n_ranks: int, exponent: float, gain: float, dtype: torch.dtype,
                             device="cpu") -> torch.Tensor:
    """x_t = g_t + gain * W_enc[:, pi(r_t)] with r_t ~ Zipf: a mean shift living in an n_ranks-dim
    subspace, which makes the pi() features far more popular than the rest."""
    d_in, d_sae = w_enc.shape
    g = normal(seed + 7919 * layer, TID_X, row0, n_rows, d_in, device)
    pi = zipf_popular_features(seed, layer, d_sae, n_ranks).to(device)
    r = zipf_ranks(seed, layer, row0, n_rows, n_ranks, exponent, device)
    dirs = w_enc.to(device)[:, pi].to(torch.float32).t().contiguous()  # [n_ranks, d_in]
    shift = dirs[r] * gain  # one rounding
    return (g + shift).to(dtype)  # one rounding, then the cast

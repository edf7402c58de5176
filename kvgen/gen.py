"""Seeded, counter-based synthetic KV pages (numpy side).

This module only makes inputs.  It holds none of the codec's arithmetic and is
the one piece that both the CPU oracle's tests and the CUDA tests/benchmark
use, so that both sides see identical bytes.  The CUDA twin (gen.cu) computes
the same function of (seed, page id, element) on the device.

Value of element k (0..2047, row-major token x channel) of page `pid`:

    c   = pid * 512 + (k >> 2)                       one 64-bit draw per 4 elements
    h   = mix64(key + c * 0x9E3779B97F4A7C15)        splitmix64 output function
    u   = (h >> (16 * (k & 3))) & 0xFFFF
    v   = fp16( table[u] * scale[row(pid)][k & 127] )   binary32 multiply, RN to binary16

`table` holds the 65,536 mid-point quantiles of N(0,1) in binary32, `scale` is a
per-(layer, K|V) vector of channel gains (outlier channels > 1), and
row(pid) = (pid // pages_per_layer) * 2 + (pid // n_kv_heads) % 2 for pages
numbered [layer][block][K|V][head].
"""
from __future__ import annotations

import numpy as np

PAGE_ELEMS = 2048
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

_table = None


def normal_table() -> np.ndarray:
    """65,536 binary32 quantiles of N(0,1) at probabilities (i + 0.5) / 65536."""
    global _table
    if _table is None:
        from scipy.special import ndtri
        p = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
        _table = ndtri(p).astype(np.float32)
    return _table


def mix64(z):
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def stream_key(seed: int) -> np.uint64:
    return mix64(np.uint64(seed & 0xFFFFFFFFFFFFFFFF) ^ np.uint64(0x5BD1E995C0FFEE11))


def scale_row(pid, pages_per_layer: int, n_kv_heads: int):
    pid = np.asarray(pid, dtype=np.uint64)
    return ((pid // np.uint64(pages_per_layer)) * np.uint64(2)
            + (pid // np.uint64(n_kv_heads)) % np.uint64(2)).astype(np.int64)


def gen_pages(seed: int, page_ids, scales: np.ndarray, pages_per_layer: int, n_kv_heads: int) -> np.ndarray:
    """Pages `page_ids` as binary16 bit patterns, shape [n, 2048] uint16."""
    pid = np.asarray(page_ids, dtype=np.uint64).reshape(-1)
    scales = np.ascontiguousarray(scales, dtype=np.float32).reshape(-1, 128)
    key = stream_key(seed)
    quad = np.arange(PAGE_ELEMS // 4, dtype=np.uint64)
    with np.errstate(over="ignore"):
        c = pid[:, None] * np.uint64(PAGE_ELEMS // 4) + quad[None, :]
        h = mix64(key + c * _GOLDEN)                                  # [n, 512]
    sh = (np.arange(4, dtype=np.uint64) * np.uint64(16))[None, None, :]
    u = ((h[:, :, None] >> sh) & np.uint64(0xFFFF)).reshape(pid.size, PAGE_ELEMS).astype(np.int64)
    rows = scale_row(pid, pages_per_layer, n_kv_heads)
    sc = scales[rows]                                                 # [n, 128]
    v = normal_table()[u] * np.tile(sc, (1, PAGE_ELEMS // 128))       # binary32 product
    return v.astype(np.float16).view(np.uint16)


def channel_scales(seed: int, n_layers: int, mode: str) -> np.ndarray:
    """Channel gains [n_layers][2][128]: row (l, 0) for K, (l, 1) for V (all ones).

    mode "fixed4":   4 outlier channels (one seeded choice for all layers), gain 10.
    mode "perlayer": per layer 2..8 outlier channels, each with its own gain in [5, 20].
    """
    sc = np.ones((n_layers, 2, 128), np.float32)
    rng = np.random.Generator(np.random.PCG64(seed ^ 0x6B766B76))
    if mode == "fixed4":
        ch = rng.choice(128, size=4, replace=False)
        sc[:, 0, ch] = 10.0
    elif mode == "perlayer":
        for l in range(n_layers):
            k = int(rng.integers(2, 9))
            ch = rng.choice(128, size=k, replace=False)
            sc[l, 0, ch] = rng.uniform(5.0, 20.0, size=k).astype(np.float32)
    else:
        raise ValueError(mode)
    return sc


RUNS_P256 = 150          # a new segment starts at a channel with probability 150/256: records of ~1,276 bytes


def runs_pages(seed: int, page_ids, p256: int = RUNS_P256) -> np.ndarray:
    """Pages whose rows are piecewise linear in the channel index, shape [n, 2048] uint16 (binary16 patterns):
    the stand-in for K/V whose consecutive differences repeat, the case the delta and run-length stages are for.

    Element (row j, channel i) of page `pid`, all integer arithmetic:

        h      = mix64(key' + (pid * 2048 + j * 128 + i) * 0x9E3779B97F4A7C15),  key' = stream_key(seed) ^ 0x52554E53
        start  = i == 0 or (h & 0xFF) < p256               a new segment begins here
        slope  = ((h >> 8) % 5) - 2 at a start, else the slope of the channel before
        u      = ((h >> 16) % 81) - 40 at i == 0 (127 in row 0), else clamp(u[i-1] + slope, -127, 127)
        value  = u / 128                                   exact in binary16; the page's largest magnitude is 127/128

    so that the quantiser's bytes are the u themselves and the delta symbols are the slopes."""
    pid = np.asarray(page_ids, dtype=np.uint64).reshape(-1)
    key = stream_key(seed) ^ np.uint64(0x52554E53)
    k = np.arange(PAGE_ELEMS, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = mix64(key + (pid[:, None] * np.uint64(PAGE_ELEMS) + k[None, :]) * _GOLDEN).reshape(pid.size, 16, 128)
    start = (h & np.uint64(0xFF)) < np.uint64(p256)
    start[:, :, 0] = True
    cand = ((h >> np.uint64(8)) % np.uint64(5)).astype(np.int64) - 2
    last = np.maximum.accumulate(np.where(start, np.arange(128)[None, None, :], 0), axis=2)
    slope = np.take_along_axis(cand, last, axis=2)
    u = np.empty((pid.size, 16, 128), np.int64)
    u[:, :, 0] = ((h[:, :, 0] >> np.uint64(16)) % np.uint64(81)).astype(np.int64) - 40
    u[:, 0, 0] = 127
    for i in range(1, 128):
        u[:, :, i] = np.clip(u[:, :, i - 1] + slope[:, :, i], -127, 127)
    return (u / 128.0).astype(np.float16).reshape(pid.size, PAGE_ELEMS).view(np.uint16)


def structured_pages(seed: int, n: int) -> np.ndarray:
    """Test-only pages with long runs: each row is made of constant-slope segments of
    geometric length (mean 8), so that consecutive differences repeat."""
    rng = np.random.Generator(np.random.PCG64(seed ^ 0x57A7))
    out = np.zeros((n, 16, 128), np.float32)
    for p in range(n):
        for j in range(16):
            i, v = 0, float(rng.integers(-40, 41))
            while i < 128:
                ln = int(min(128 - i, rng.geometric(1.0 / 8.0)))
                slope = float(rng.integers(-2, 3))
                out[p, j, i:i + ln] = v + slope * np.arange(ln)
                v = out[p, j, i + ln - 1]
                i += ln
        out[p] *= 127.0 / max(1.0, float(np.abs(out[p]).max()))
    return (out / 127.0).astype(np.float16).reshape(n, PAGE_ELEMS).view(np.uint16)

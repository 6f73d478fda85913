"""Seeded synthetic inputs for the GPTQ layer solver (host side, numpy).

This module holds no arithmetic of the quantization method: it only produces
the weight matrices W and calibration activations X that both the CUDA path and
the CPU oracle are fed.  Everything is counter based -- element (row, col) of a
tensor is a pure function of (stream seed, flat index) -- so any row range,
column subset or single element can be produced on its own, in any order, and a
device-side filler can reproduce the same bits.

Recipe (stands in for trained OPT/BLOOM weights and C4 activations, which are
not available offline):

* W[r, c]  = fp16_rne(0.02 * z)                       (std 0.02)
* X[t, c]  = bf16_rne(z * s[c])                       (tokens x channels)
* s[c]     = exp(z_c) (log-normal(0, 1)), times 20 for max(1, round(0.005 C))
             outlier channels chosen by a seeded ranking
* z        = standard normal from a 64-bit counter hash: the top 16 bits pick a
             cell of a 65537-entry fp32 quantile table, the next 24 bits
             interpolate linearly inside the cell.  Only IEEE fp32 add, sub and
             mul (no fused multiply-add) are used after the table lookup, so a
             GPU filler that uses the same table is bit-identical.
"""
from __future__ import annotations

import functools

import numpy as np

BASE_SEED = 221017323
GENERATOR_VERSION = 1

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)

TENSOR_W = 1
TENSOR_X = 2
TENSOR_SCALES = 3
TENSOR_OUTLIERS = 4


def mix64(z):
    """splitmix64 finalizer on uint64 (wrapping arithmetic)."""
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _C1
        z = (z ^ (z >> np.uint64(27))) * _C2
        z = z ^ (z >> np.uint64(31))
    return z


def stream_seed(config_id: int, block_idx: int, layer_kind: int, tensor_kind: int,
                base: int = BASE_SEED) -> int:
    """One 64-bit seed per (config, block, layer kind, tensor kind)."""
    s = np.uint64(base)
    with np.errstate(over="ignore"):
        for v in (config_id, block_idx, layer_kind, tensor_kind):
            s = mix64(s * _GOLD + np.uint64(v) + np.uint64(1))
    return int(s)


def counter_hash(seed: int, idx) -> np.ndarray:
    """64 random bits for flat index idx of stream seed."""
    idx = np.asarray(idx, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return mix64(np.uint64(seed) ^ (idx * _GOLD))


@functools.lru_cache(maxsize=1)
def normal_table() -> np.ndarray:
    """fp32 table T[k] = Phi^-1(k / 65536), k = 0..65536, tails clipped at 2^-21.

    Built with Acklam's rational approximation followed by one Newton step on
    erfc, all in fp64 with numpy only, then rounded to fp32.  The same array is
    uploaded to the device for the GPU filler, so host and device always agree.
    """
    import math

    k = np.arange(65537, dtype=np.float64)
    p = k / 65536.0
    p[0] = 2.0 ** -21
    p[-1] = 1.0 - 2.0 ** -21
    a = [-3.969683028665376e+01, 2.209460984245205e+02, -2.759285104469687e+02,
         1.383577518672690e+02, -3.066479806614716e+01, 2.506628277459239e+00]
    b = [-5.447609879822406e+01, 1.615858368580409e+02, -1.556989798598866e+02,
         6.680131188771972e+01, -1.328068155288572e+01]
    c = [-7.784894002430293e-03, -3.223964580411365e-01, -2.400758277161838e+00,
         -2.549732539343734e+00, 4.374664141464968e+00, 2.938163982698783e+00]
    d = [7.784695709041462e-03, 3.224671290700398e-01, 2.445134137142996e+00,
         3.754408661907416e+00]
    x = np.empty_like(p)
    lo = p < 0.02425
    hi = p > 1 - 0.02425
    mid = ~(lo | hi)
    q = np.sqrt(-2 * np.log(p[lo]))
    x[lo] = (((((c[0] * q + c[1]) * q + c[2]) * q + c[3]) * q + c[4]) * q + c[5]) / \
            ((((d[0] * q + d[1]) * q + d[2]) * q + d[3]) * q + 1)
    q = np.sqrt(-2 * np.log(1 - p[hi]))
    x[hi] = -(((((c[0] * q + c[1]) * q + c[2]) * q + c[3]) * q + c[4]) * q + c[5]) / \
            ((((d[0] * q + d[1]) * q + d[2]) * q + d[3]) * q + 1)
    q = p[mid] - 0.5
    r = q * q
    x[mid] = (((((a[0] * r + a[1]) * r + a[2]) * r + a[3]) * r + a[4]) * r + a[5]) * q / \
             (((((b[0] * r + b[1]) * r + b[2]) * r + b[3]) * r + b[4]) * r + 1)
    erfc = np.vectorize(math.erfc)
    for _ in range(2):  # Newton polish
        e = 0.5 * erfc(-x / math.sqrt(2.0)) - p
        x = x - e * math.sqrt(2.0 * math.pi) * np.exp(0.5 * x * x)
    x[32768] = 0.0
    t = x.astype(np.float32)
    t.setflags(write=False)
    return t


def std_normal(seed: int, idx) -> np.ndarray:
    """fp32 standard-normal variates for flat indices idx (any shape)."""
    h = counter_hash(seed, idx)
    t = normal_table()
    k = (h >> np.uint64(48)).astype(np.int64)
    frac = ((h >> np.uint64(24)) & np.uint64(0xFFFFFF)).astype(np.float32) * np.float32(2.0 ** -24)
    t0 = t[k]
    d = (t[k + 1] - t0).astype(np.float32)
    p = (d * frac).astype(np.float32)
    return (t0 + p).astype(np.float32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def channel_scales(seed_scales: int, seed_outliers: int, C: int) -> np.ndarray:
    """fp32 per-channel scale s[c]: log-normal(0,1), 0.5 % of channels times 20."""
    z = std_normal(seed_scales, np.arange(C, dtype=np.uint64)).astype(np.float64)
    s = np.exp(z)
    n_out = max(1, int(round(0.005 * C)))
    rank = counter_hash(seed_outliers, np.arange(C, dtype=np.uint64))
    chosen = np.argsort(rank, kind="stable")[:n_out]
    s[chosen] *= 20.0
    return s.astype(np.float32)


def gen_x_bits(seed: int, scales: np.ndarray, C: int, t0: int, t1: int, cols=None) -> np.ndarray:
    """bf16 bit patterns of X[t0:t1, cols] (tokens x channels, row-major)."""
    cols = np.arange(C, dtype=np.uint64) if cols is None else np.asarray(cols, dtype=np.uint64)
    t = np.arange(t0, t1, dtype=np.uint64)[:, None]
    idx = t * np.uint64(C) + cols[None, :]
    z = std_normal(seed, idx)
    v = (z * scales[cols.astype(np.int64)][None, :].astype(np.float32)).astype(np.float32)
    return f32_to_bf16_bits(v)


def gen_w(seed: int, R: int, C: int, rows=None) -> np.ndarray:
    """fp16 W[rows, :] with std 0.02 (rows=None: all R rows)."""
    rows = np.arange(R, dtype=np.uint64) if rows is None else np.asarray(rows, dtype=np.uint64)
    idx = rows[:, None] * np.uint64(C) + np.arange(C, dtype=np.uint64)[None, :]
    z = std_normal(seed, idx)
    return (z * np.float32(0.02)).astype(np.float32).astype(np.float16)

"""fp64 CPU oracle for the GPTQ layer solver.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this file.  It shares no code with the CUDA path and never imports it.  It is
written for readability, not speed: every function takes the paper's steps in
the paper's order and notation, in double precision, with numpy/LAPACK
primitives (matmul, Cholesky, triangular solve) as single steps and no
blocking or reordering beyond what the cited passage states.

Notation: W is d_row x d_col (R x C).  The paper's X is d_col x m; inputs here
arrive as the transposed, token-major array Xt (m x C).  H = 2 X X^T.
U is the upper-triangular matrix Algorithm 1 calls "Cholesky(H^-1)^T".

Pins (tests/test_oracle_pins.py): diagonal H reduces to round-to-nearest;
group grids equal the min-max grid of the trajectory-reconstructed current weights;
block-size invariance; equivalence with the sequential OBQ recursion (Eq. 2,
Eq. 3) for d_col <= 16; exhaustive search on d_col <= 8 at 2 bits never beaten;
loss identity sum(E^2) = 2||dW X||^2 + lambda ||dW||^2; 2x2 closed form of U;
integer-exact Hessians; hand-worked packed words; power-of-two scale invariance.

Parity unpinned by the paper (pinned only through the general pins above): the
symmetric grid and the ternary grid's scale choice -- the paper states neither.
"""
from __future__ import annotations

import numpy as np
import scipy.linalg

BITS_TERNARY = -1


# --------------------------------------------------------------------------- inputs
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact promotion of bf16 bit patterns (uint16) to float64."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------- stage 1
def hessian_accumulate(H: np.ndarray, Xt_bits: np.ndarray, chunk: int = 4096) -> np.ndarray:
    """H += 2 X X^T  (Section 2, "Optimal Brain Quantization": H_F = 2 X_F X_F^T;
    Algorithm 1 caption).  Plain sum over tokens, no 1/m factor.  Xt_bits is
    (tokens x C) bf16 bit patterns; tokens are consumed in chunks only to bound
    memory (the sum is the same)."""
    n = Xt_bits.shape[0]
    for t0 in range(0, n, chunk):
        Xt = bf16_bits_to_f64(Xt_bits[t0:t0 + chunk])
        H += 2.0 * (Xt.T @ Xt)
    return H


# --------------------------------------------------------------------------- stage 2
def dampen(H: np.ndarray, damp: float) -> tuple[np.ndarray, float]:
    """H~ = H + lambda I with lambda = damp x the mean of H's diagonal (Section 3, Step 3; the
    paper's setting is damp = 0.01)."""
    lam = float(damp) * float(np.mean(np.diag(H)))
    Ht = H.copy()
    Ht[np.diag_indices_from(Ht)] += lam
    return Ht, lam


def cholesky_inverse_upper(Ht: np.ndarray) -> np.ndarray:
    """U = Cholesky(H~^-1)^T, upper triangular, positive diagonal, U^T U = H~^-1
    (Algorithm 1, third line).  Literal route: factor H~, invert through the
    factor, factor the inverse, transpose.  Raises LinAlgError if H~ is not
    positive definite."""
    L = np.linalg.cholesky(Ht)                                   # H~ = L L^T
    Linv = scipy.linalg.solve_triangular(L, np.eye(Ht.shape[0]), lower=True)
    Hinv = Linv.T @ Linv                                         # H~^-1
    L2 = np.linalg.cholesky(Hinv)                                # H~^-1 = L2 L2^T
    return np.ascontiguousarray(L2.T)                            # U = L2^T


# --------------------------------------------------------------------------- grid
def maxq_of(bits: int) -> int:
    """Largest code: 2^b - 1; the ternary grid {-1, 0, +1} x scale has codes 0, 1, 2."""
    return 2 if bits == BITS_TERNARY else (1 << bits) - 1


def field_bits_of(bits: int) -> int:
    """Width of one packed code; ternary codes are stored in 2-bit fields."""
    return 2 if bits == BITS_TERNARY else bits


def _storage_rounded(scale: np.ndarray, scale_fp16: bool) -> np.ndarray:
    """The scale in the precision it is returned (and, with scale_fp16, stored) in, as float64 values.
    fp32 always; with scale_fp16 additionally rounded to the nearest fp16 value (Section 5, Extreme Quantization,
    counts one FP16 scale per group) unless that would be 0 or infinite, in which case the fp32 value stays."""
    s32 = scale.astype(np.float32)
    if not scale_fp16:
        return s32.astype(np.float64)
    with np.errstate(over="ignore"):
        s16 = s32.astype(np.float16)
    usable = np.isfinite(s16) & (s16 > 0)
    return np.where(usable, s16.astype(np.float64), s32.astype(np.float64))


def find_params(v: np.ndarray, bits: int, sym: bool, scale_fp16: bool = False):
    """Min-max grid of each row of v (Section 5, Setup: asymmetric uniform grid spanning the
    row's minimum and maximum; grouping applies the same to g consecutive weights).
    The range is widened to contain 0 so the zero-point is an integer code (Section 5,
    Extreme Quantization, counts a b-bit zero-point per group in its storage figures).  An
    all-zero row gets [-1, 1].  Symmetric / ternary: half-range a = max|v|,
    scale = 2a/maxq, zero = (maxq+1)//2.  The scale is rounded to fp32 -- the
    precision it is returned in -- and used as that value; with scale_fp16 it is rounded to
    fp16 instead (the stored model's precision), BEFORE the zero-point is derived from it.
    Returns (scale[R] float64 holding fp32 values, zero[R] float64 holding integers)."""
    maxq = maxq_of(bits)
    xmin = np.minimum(v.min(axis=1), 0.0)
    xmax = np.maximum(v.max(axis=1), 0.0)
    dead = (xmin == 0.0) & (xmax == 0.0)
    xmin = np.where(dead, -1.0, xmin)
    xmax = np.where(dead, 1.0, xmax)
    if sym or bits == BITS_TERNARY:
        a = np.maximum(np.abs(xmin), xmax)
        scale = _storage_rounded(2.0 * a / maxq, scale_fp16)
        zero = np.full_like(scale, float((maxq + 1) // 2))
    else:
        scale = _storage_rounded((xmax - xmin) / maxq, scale_fp16)
        zero = np.rint(-xmin / scale)
    return scale, zero


def quant(w: np.ndarray, scale: np.ndarray, zero: np.ndarray, maxq: int):
    """quant(w): nearest grid value (Section 2).  Code q = clamp(rne(w/scale) + zero,
    0, maxq); value = scale * (q - zero).  Ties round half to even."""
    q = np.clip(np.rint(w / scale) + zero, 0.0, float(maxq))
    return q, scale * (q - zero)


# --------------------------------------------------------------------------- stage 3
def _fix_group_grid(W, j, g, bits, sym, scales, zeros, scale_fp16=False):
    """Column j opens a group: its g columns, in the state the error feedback of all earlier
    columns has left them, decide the group's scale and zero-point (Section 5, grouping)."""
    scales[:, j // g], zeros[:, j // g] = find_params(W[:, j:j + g], bits, sym, scale_fp16)


def _round_column_and_feed_back(W, U, j, stop, s, z, maxq):
    """Algorithm 1, one pass of the inner loop for column j (all rows at once): pick the grid
    point, form the scaled error (w - quant(w)) / U_jj, and subtract error x U[j, j:stop] from
    columns j .. stop-1 (which also sets column j itself to its grid point).
    Returns (codes, grid values, scaled errors) of the column."""
    q, wq = quant(W[:, j], s, z, maxq)
    err = (W[:, j] - wq) / U[j, j]
    W[:, j:stop] -= np.outer(err, U[j, j:stop])
    return q.astype(np.int32), wq, err


def _push_block_errors(W, U, E, i, stop):
    """Algorithm 1, last line of the outer loop: the block's errors reach every later column in
    one product, W[:, stop:] -= E U[i:stop, stop:] (the lazy batch update of Section 3, Step 2)."""
    W[:, stop:] -= E @ U[i:stop, stop:]


def quantize_layer(W16: np.ndarray, U: np.ndarray, bits: int, group_size: int = 0,
                   sym: bool = False, block: int = 128, scale_fp16: bool = False):
    """Algorithm 1 with lazy batch updates of `block` columns.

    W16: (R x C) fp16 (promoted exactly to double); U: (C x C) upper factor.
    One grid per row (group_size <= 0): decided once from the untouched row, before any column
    is processed (Section 2 takes the grid as given in advance).  Grouped: decided per group
    when its first column is reached, from the weights as updated up to then (Section 5).
    Returns dict(codes int32 RxC, scales RxG, zeros RxG, loss, W_hat RxC, E RxC)."""
    W = np.asarray(W16, dtype=np.float64).copy()
    R, C = W.shape
    maxq = maxq_of(bits)
    grouped = group_size > 0
    g = group_size if grouped else C
    if C % g != 0:
        raise ValueError("group size must divide d_col")
    if grouped and g % block != 0 and block % g != 0:
        # a group cut by a block end would see some of its columns before and some after the
        # lazy update; only nested groups and blocks give "the weights as updated so far" a meaning
        raise ValueError("group size and block size must nest")
    G = C // g
    W_hat = np.zeros((R, C))
    codes = np.zeros((R, C), dtype=np.int32)
    scales = np.zeros((R, G))
    zeros = np.zeros((R, G))
    E_all = np.zeros((R, C))
    if not grouped:
        scales[:, 0], zeros[:, 0] = find_params(W, bits, sym, scale_fp16)
    for i in range(0, C, block):
        stop = min(i + block, C)
        E = np.zeros((R, stop - i))
        for j in range(i, stop):
            if grouped and j % g == 0:
                _fix_group_grid(W, j, g, bits, sym, scales, zeros, scale_fp16)
            codes[:, j], W_hat[:, j], E[:, j - i] = _round_column_and_feed_back(
                W, U, j, stop, scales[:, j // g], zeros[:, j // g], maxq)
        _push_block_errors(W, U, E, i, stop)
        E_all[:, i:stop] = E
    loss = float(np.sum(E_all * E_all))
    return dict(codes=codes, scales=scales, zeros=zeros, loss=loss, W_hat=W_hat, E=E_all)


def rtn(W16: np.ndarray, bits: int, group_size: int = 0, sym: bool = False, scale_fp16: bool = False):
    """Round-to-nearest on the same grid, no error feedback (Section 5, Baselines)."""
    W = np.asarray(W16, dtype=np.float64)
    R, C = W.shape
    g = group_size if group_size > 0 else C
    codes = np.zeros((R, C), dtype=np.int32)
    What = np.zeros((R, C))
    for j0 in range(0, C, g):
        s, z = find_params(W[:, j0:j0 + g], bits, sym, scale_fp16)
        q, What[:, j0:j0 + g] = quant(W[:, j0:j0 + g], s[:, None], z[:, None], maxq_of(bits))
        codes[:, j0:j0 + g] = q.astype(np.int32)
    return codes, What


def reconstruction_error(W16: np.ndarray, W_hat: np.ndarray, H: np.ndarray) -> float:
    """||W X - W^ X||_F^2 of Eq. 1, evaluated through the undamped H = 2 X X^T:
    ||dW X||^2 = tr(dW X X^T dW^T) = 0.5 tr(dW H dW^T)."""
    dW = np.asarray(W16, dtype=np.float64) - W_hat
    return 0.5 * float(np.sum((dW @ H) * dW))


# --------------------------------------------------------------------------- packing
def pack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """Packed layout (defined by this library; the paper is silent): per row a
    little-endian bit stream, code of column c in stream bits [c f, c f + f),
    f = field width; uint32 word k holds stream bits [32k, 32k+32)."""
    f = field_bits_of(bits)
    R, C = codes.shape
    if C % 32 != 0:
        raise ValueError("d_col must be a multiple of 32")
    nwords = C * f // 32
    out = np.zeros((R, nwords), dtype=np.uint64)
    for c in range(C):
        v = codes[:, c].astype(np.uint64)
        bit = c * f
        k, o = divmod(bit, 32)
        out[:, k] |= (v << np.uint64(o)) & np.uint64(0xFFFFFFFF)
        if o + f > 32:
            out[:, k + 1] |= v >> np.uint64(32 - o)
    return out.astype(np.uint32)


def unpack_codes(words: np.ndarray, bits: int, C: int) -> np.ndarray:
    f = field_bits_of(bits)
    R = words.shape[0]
    w = words.astype(np.uint64)
    out = np.zeros((R, C), dtype=np.int32)
    mask = np.uint64((1 << f) - 1)
    for c in range(C):
        k, o = divmod(c * f, 32)
        v = w[:, k] >> np.uint64(o)
        if o + f > 32:
            v |= w[:, k + 1] << np.uint64(32 - o)
        out[:, c] = (v & mask).astype(np.int32)
    return out


# --------------------------------------------------------------------------- using the packed weights
def dequantize(codes: np.ndarray, scales: np.ndarray, zeros: np.ndarray, to_fp16: bool = False) -> np.ndarray:
    """W^ = scale * (code - zero) per row and group (Section 5, Extreme Quantization: one scale and one zero-point per group).
    to_fp16=False: the exact real-valued grid point in float64 (scales hold fp32 values).
    to_fp16=True: the stored-model reading -- one fp32 multiply, then round-to-nearest-even to fp16."""
    R, C = codes.shape
    g = C // scales.shape[1]
    s = np.repeat(scales, g, axis=1)
    z = np.repeat(zeros, g, axis=1)
    if not to_fp16:
        return s.astype(np.float64) * (codes.astype(np.float64) - z.astype(np.float64))
    d = (codes.astype(np.float32) - z.astype(np.float32)).astype(np.float32)
    return (s.astype(np.float32) * d).astype(np.float32).astype(np.float16)


def matvec(codes: np.ndarray, scales: np.ndarray, zeros: np.ndarray, x16: np.ndarray) -> np.ndarray:
    """y = W^ x for one input vector (Section 5, Practical Speedups: quantized-matrix times
    full-precision vector), in float64 on the exact grid values."""
    return dequantize(codes, scales, zeros) @ np.asarray(x16, dtype=np.float64)


# --------------------------------------------------------------------------- whole path
def solve_layer(W16, Xt_bits, bits, group_size=0, sym=False, block=128, damp=0.01):
    """Stages 1-3 in sequence; returns the stage-3 dict plus H, U, lambda."""
    C = W16.shape[1]
    H = hessian_accumulate(np.zeros((C, C)), Xt_bits)
    Ht, lam = dampen(H, damp)
    U = cholesky_inverse_upper(Ht)
    out = quantize_layer(W16, U, bits, group_size, sym, block)
    out.update(H=H, U=U, lam=lam)
    return out

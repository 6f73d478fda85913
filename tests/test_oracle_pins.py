"""Pins for the fp64 oracle: what the paper and the mathematics fix, independent of the oracle.

Each test names the passage it rests on.  None of them re-types the oracle's own
formulas: they use brute force, closed forms, the sequential OBQ recursion, or
exact integer arithmetic instead.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import gptq_oracle as O

RNG = np.random.default_rng


def _bf16_bits(x):
    """Round float array to bf16 bits (test-side helper, round-to-nearest-even)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def _random_problem(R, C, m, seed, scale_spread=True):
    r = RNG(seed)
    s = np.exp(r.normal(size=C)) if scale_spread else np.ones(C)
    Xt = _bf16_bits(r.normal(size=(m, C)) * s)
    W = (r.normal(size=(R, C)) * 0.02).astype(np.float16)
    return W, Xt


def _grid_values(scale, zero, maxq):
    return [scale * (q - zero) for q in range(maxq + 1)]


def _nearest_code_bruteforce(w, scale, zero, maxq):
    """Definition of quant(): the nearest grid value, by trying every level."""
    vals = np.array(_grid_values(scale, zero, maxq))
    return int(np.argmin(np.abs(vals - w)))


# ------------------------------------------------------------------ stage 1 (Section 2: H = 2 X X^T)
def test_hessian_integer_exact_and_additive():
    r = RNG(1)
    m, C = 300, 40
    Xi = r.integers(-8, 9, size=(m, C))
    bits = _bf16_bits(Xi.astype(np.float32))
    H = O.hessian_accumulate(np.zeros((C, C)), bits)
    exact = 2 * (Xi.T.astype(np.int64) @ Xi.astype(np.int64))
    assert np.array_equal(H, exact.astype(np.float64))
    # additive over any chunking of the tokens (Section 5 Setup: Hessians are summed over batches)
    H2 = np.zeros((C, C))
    for a, b in ((0, 7), (7, 128), (128, 300)):
        O.hessian_accumulate(H2, bits[a:b])
    assert np.array_equal(H, H2)
    # diagonal: H_jj = 2 sum_t x_tj^2 ; symmetric; PSD
    assert np.array_equal(np.diag(H), 2.0 * (Xi.astype(np.float64) ** 2).sum(0))
    assert np.array_equal(H, H.T)
    assert np.linalg.eigvalsh(H).min() > -1e-9


def test_hessian_single_token_outer_product():
    x = np.array([[1.5, -2.0, 0.25]], dtype=np.float32)
    H = O.hessian_accumulate(np.zeros((3, 3)), _bf16_bits(x))
    want = [[4.5, -6.0, 0.75], [-6.0, 8.0, -1.0], [0.75, -1.0, 0.125]]
    assert np.array_equal(H, np.array(want))


# ------------------------------------------------------------------ stage 2 (Section 3 Step 3; Algorithm 1)
def test_dampen_is_one_percent_of_mean_diagonal():
    H = np.diag([1.0, 2.0, 3.0, 10.0]) + 0.1
    Ht, lam = O.dampen(H, 0.01)
    assert lam == pytest.approx(0.01 * (1.1 + 2.1 + 3.1 + 10.1) / 4)
    assert np.allclose(Ht - H, lam * np.eye(4))


def test_U_2x2_closed_form():
    a, b, c = 3.0, 0.7, 2.0
    Ht = np.array([[a, b], [b, c]])
    D = a * c - b * b
    want = np.array([[np.sqrt(c / D), -b / np.sqrt(D * c)], [0.0, 1.0 / np.sqrt(c)]])
    assert np.allclose(O.cholesky_inverse_upper(Ht), want, rtol=1e-13, atol=0)


def test_U_properties_and_reverse_route():
    W, Xt = _random_problem(4, 48, 400, 2)
    H = O.hessian_accumulate(np.zeros((48, 48)), Xt)
    Ht, _ = O.dampen(H, 0.01)
    U = O.cholesky_inverse_upper(Ht)
    assert np.array_equal(U, np.triu(U)) and (np.diag(U) > 0).all()
    assert np.allclose(U.T @ U @ Ht, np.eye(48), atol=1e-9)
    # last diagonal entry: U_CC = H~_CC^{-1/2}
    assert U[-1, -1] == pytest.approx(Ht[-1, -1] ** -0.5, rel=1e-12)
    # the same U by another route: factor H~ = Ut Ut^T with Ut upper (Cholesky of the
    # index-reversed matrix), then invert -- unique upper factor with positive diagonal
    J = np.eye(48)[::-1]
    L = np.linalg.cholesky(J @ Ht @ J)
    Ut = J @ L @ J
    assert np.allclose(Ut @ Ut.T, Ht, rtol=1e-12)
    assert np.allclose(np.linalg.inv(Ut), U, rtol=1e-8, atol=1e-12)


def test_U_diagonal_H_closed_form():
    d = np.array([4.0, 1.0, 0.25, 9.0])
    U = O.cholesky_inverse_upper(np.diag(d))
    assert np.allclose(U, np.diag(d ** -0.5), rtol=1e-14)


def test_not_positive_definite_raises():
    with pytest.raises(np.linalg.LinAlgError):
        O.cholesky_inverse_upper(np.array([[1.0, 2.0], [2.0, 1.0]]))


# ------------------------------------------------------------------ grid (Section 5 Setup; Extreme Quantization)
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_minmax_grid_endpoints_and_integer_zero(bits):
    r = RNG(3)
    v = r.normal(size=(50, 64)) * 0.02
    v[0] = np.abs(v[0])          # all-positive row: range must still contain 0
    v[1] = -np.abs(v[1])         # all-negative row
    v[2] = 0.0                   # dead row
    s, z = O.find_params(v, bits, sym=False)
    maxq = 2 ** bits - 1
    assert (z == np.rint(z)).all() and (z >= 0).all() and (z <= maxq).all()
    assert (s == s.astype(np.float32)).all() and (s > 0).all()
    lo, hi = s * (0 - z), s * (maxq - z)
    # grid spans the row's range widened to 0, to within one rounding of the zero-point (half a step)
    assert (lo <= np.minimum(v.min(1), 0) + 0.5 * s * (1 + 1e-6)).all()
    assert (hi >= np.maximum(v.max(1), 0) - 0.5 * s * (1 + 1e-6)).all()
    assert z[0] == 0 and z[1] == maxq
    # zero is exactly representable: quantizing 0 gives 0
    q, val = O.quant(np.zeros(50), s, z, maxq)
    assert (val == 0).all()


def test_quant_is_nearest_grid_value_bruteforce():
    r = RNG(4)
    for bits in (2, 3, 4):
        maxq = 2 ** bits - 1
        v = r.normal(size=(20, 32)) * 0.02
        s, z = O.find_params(v, bits, sym=False)
        w = r.normal(size=(20, 200)) * 0.03          # includes out-of-range values (clamped)
        q, val = O.quant(w, s[:, None], z[:, None], maxq)
        for i in range(20):
            for j in range(0, 200, 7):
                assert int(q[i, j]) == _nearest_code_bruteforce(w[i, j], s[i], z[i], maxq)
                assert val[i, j] == s[i] * (q[i, j] - z[i])


def test_ternary_and_symmetric_grids():
    v = np.array([[0.5, -1.0, 0.25, 0.9], [0.1, 0.2, 0.3, 0.0]])
    s, z = O.find_params(v, O.BITS_TERNARY, sym=False)
    assert list(s) == [1.0, np.float64(np.float32(0.3))] and list(z) == [1.0, 1.0]
    q, val = O.quant(v, s[:, None], z[:, None], 2)
    assert q[0].tolist() == [1, 0, 1, 2] or q[0].tolist() == [2, 0, 1, 2]   # 0.5 is a tie: either level is nearest
    assert set(np.unique(val[0] / s[0])) <= {-1.0, 0.0, 1.0}
    s4, z4 = O.find_params(v, 4, sym=True)
    assert z4.tolist() == [8.0, 8.0] and s4[0] == np.float64(np.float32(2.0 / 15))


# ------------------------------------------------------------------ P1: diagonal H => RTN (Section 5, Baselines)
@pytest.mark.parametrize("bits,group", [(4, 0), (3, 0), (2, 16), (O.BITS_TERNARY, 16), (3, 32)])
def test_diagonal_hessian_reduces_to_rtn(bits, group):
    r = RNG(5)
    R, C = 24, 64
    W = (r.normal(size=(R, C)) * 0.02).astype(np.float16)
    d = np.exp(r.normal(size=C))
    Ht, lam = O.dampen(np.diag(d), 0.01)
    U = O.cholesky_inverse_upper(Ht)
    assert np.allclose(U, np.diag((d + lam) ** -0.5), rtol=1e-13)
    out = O.quantize_layer(W, U, bits, group, False, block=16)
    # RTN by definition: nearest level, every weight on its own, grid from the ORIGINAL weights
    Wd = W.astype(np.float64)
    g = group if group > 0 else C
    maxq = O.maxq_of(bits)
    for rr in range(R):
        for c in range(C):
            s, z = out["scales"][rr, c // g], out["zeros"][rr, c // g]
            vals = np.array(_grid_values(s, z, maxq))
            dist = np.abs(vals - Wd[rr, c])
            assert dist[out["codes"][rr, c]] == dist.min()
    codes_rtn, _ = O.rtn(W, bits, group, False)
    assert np.array_equal(codes_rtn, out["codes"])
    # and the grid is the original weights' min-max grid (no update ever touched them)
    for gi in range(C // g):
        seg = Wd[:, gi * g:(gi + 1) * g]
        lo, hi = np.minimum(seg.min(1), 0), np.maximum(seg.max(1), 0)
        if bits != O.BITS_TERNARY:
            assert np.allclose(out["scales"][:, gi], (hi - lo) / maxq, rtol=1e-6)


# ------------------------------------------------------------------ P2: block-size invariance (Section 3, Step 2)
@pytest.mark.parametrize("bits,group", [(4, 0), (3, 32), (2, 32), (O.BITS_TERNARY, 32)])
def test_block_size_invariance(bits, group):
    W, Xt = _random_problem(16, 96, 500, 6)
    H = O.hessian_accumulate(np.zeros((96, 96)), Xt)
    U = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0])
    ref = O.quantize_layer(W, U, bits, group, False, block=1)
    for B in (32, 96, 128) + ((8, 16) if group else (7, 50)):
        if group and (B % group and group % B):
            continue
        out = O.quantize_layer(W, U, bits, group, False, block=B)
        assert np.array_equal(out["codes"], ref["codes"]), B
        assert np.array_equal(out["scales"], ref["scales"]) and np.array_equal(out["zeros"], ref["zeros"])
        assert out["loss"] == pytest.approx(ref["loss"], rel=1e-10)


def test_group_block_must_nest():
    W, Xt = _random_problem(2, 96, 200, 7)
    U = np.eye(96)
    with pytest.raises(ValueError):
        O.quantize_layer(W, U, 4, 32, False, block=48)


# ------------------------------------------------------------------ P3: sequential OBQ with fixed order (Eq. 2, Eq. 3)
def _obq_fixed_order(w, Hinv, scale, zero, maxq):
    """One row, columns in natural order: quantize w_q, apply the optimal update of
    Eq. 2 to the remaining weights, remove q from the inverse with Eq. 3."""
    w = w.copy()
    Hinv = Hinv.copy()
    C = len(w)
    alive = list(range(C))
    codes = np.zeros(C, dtype=np.int64)
    rows = []
    for q in range(C):
        loc = alive.index(q)
        rows.append(Hinv[loc, loc:].copy())
        code = _nearest_code_bruteforce(w[q], scale, zero, maxq)
        codes[q] = code
        wq = scale * (code - zero)
        delta = -(w[q] - wq) / Hinv[loc, loc] * Hinv[:, loc]
        for a, col in enumerate(alive):
            w[col] += delta[a]
        assert abs(w[q] - wq) < 1e-12
        Hinv = Hinv - np.outer(Hinv[:, loc], Hinv[loc, :]) / Hinv[loc, loc]
        Hinv = np.delete(np.delete(Hinv, loc, 0), loc, 1)
        alive.pop(loc)
    return codes, rows


@pytest.mark.parametrize("C,bits", [(5, 3), (12, 4), (16, 2)])
def test_cholesky_form_equals_sequential_obq(C, bits):
    W, Xt = _random_problem(6, C, 80, 8 + C)
    H = O.hessian_accumulate(np.zeros((C, C)), Xt)
    Ht, _ = O.dampen(H, 0.01)
    U = O.cholesky_inverse_upper(Ht)
    out = O.quantize_layer(W, U, bits, 0, False, block=4)
    Hinv = np.linalg.inv(Ht)
    for r in range(W.shape[0]):
        codes, rows = _obq_fixed_order(W[r].astype(np.float64), Hinv, out["scales"][r, 0],
                                       out["zeros"][r, 0], 2 ** bits - 1)
        assert np.array_equal(codes, out["codes"][r])
        # row q of the running inverse, from the diagonal on, equals U_qq * U[q, q:]  (Step 3)
        for q in range(C):
            assert np.allclose(rows[q], U[q, q] * U[q, q:], rtol=1e-8, atol=1e-14)


# ------------------------------------------------------------------ P4: exhaustive search never beaten (Eq. 1)
@pytest.mark.parametrize("C", [1, 4, 7])
def test_greedy_never_beats_exhaustive(C):
    bits, maxq = 2, 3
    W, Xt = _random_problem(5, C, 60, 20 + C)
    H = O.hessian_accumulate(np.zeros((C, C)), Xt)
    Ht, lam = O.dampen(H, 0.01)
    U = O.cholesky_inverse_upper(Ht)
    out = O.quantize_layer(W, U, bits, 0, False, block=3)
    for r in range(W.shape[0]):
        w = W[r].astype(np.float64)
        s, z = out["scales"][r, 0], out["zeros"][r, 0]
        vals = np.array(_grid_values(s, z, maxq))
        best = np.inf
        for assign in itertools.product(range(maxq + 1), repeat=C):
            d = w - vals[list(assign)]
            best = min(best, d @ Ht @ d)
        dg = w - out["W_hat"][r]
        greedy = dg @ Ht @ dg
        assert greedy >= best * (1 - 1e-12)
        if C == 1:
            assert greedy == pytest.approx(best, rel=1e-12)
        # the per-row loss the solver reports is that same quadratic form
        assert np.sum(out["E"][r] ** 2) == pytest.approx(greedy, rel=1e-9)


# ------------------------------------------------------------------ P5: loss identity along any trajectory
@pytest.mark.parametrize("bits,group", [(4, 0), (2, 16)])
def test_loss_identity_against_direct_reconstruction(bits, group):
    W, Xt = _random_problem(10, 64, 300, 9)
    X = O.bf16_bits_to_f64(Xt).T                       # C x m, the paper's orientation
    H = O.hessian_accumulate(np.zeros((64, 64)), Xt)
    Ht, lam = O.dampen(H, 0.01)
    U = O.cholesky_inverse_upper(Ht)
    out = O.quantize_layer(W, U, bits, group, False, block=16)
    dW = W.astype(np.float64) - out["W_hat"]
    direct = np.sum((dW @ X) ** 2)                     # ||W X - W^ X||_F^2, Eq. 1, straight from X
    assert out["loss"] == pytest.approx(2 * direct + lam * np.sum(dW ** 2), rel=1e-9)
    assert O.reconstruction_error(W, out["W_hat"], H) == pytest.approx(direct, rel=1e-10)
    # W0 - W^ = E U exactly
    assert np.allclose(out["E"] @ U, dW, rtol=1e-9, atol=1e-15)


def test_error_feedback_beats_rtn_on_correlated_inputs():
    """The point of the method (Section 5, Baselines: same grid, direct rounding): with
    strongly correlated input channels the compensated solution has a much smaller
    layer error (Eq. 1) than round-to-nearest on the same grid."""
    r = RNG(14)
    C, m = 64, 400
    Z = r.normal(size=(m, 8)) @ r.normal(size=(8, C)) + 0.05 * r.normal(size=(m, C))
    Xt = _bf16_bits(Z)
    W = (r.normal(size=(10, C)) * 0.02).astype(np.float16)
    H = O.hessian_accumulate(np.zeros((C, C)), Xt)
    U = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0])
    out = O.quantize_layer(W, U, 4, 0, False, block=16)
    _, What_rtn = O.rtn(W, 4, 0, False)
    assert O.reconstruction_error(W, out["W_hat"], H) < 0.5 * O.reconstruction_error(W, What_rtn, H)


# ------------------------------------------------------------------ grouped grids come from the UPDATED weights (Section 5)
@pytest.mark.parametrize("bits,group,block", [(4, 16, 16), (3, 16, 32), (2, 32, 16), (3, 8, 64)])
def test_group_grid_is_taken_from_current_weights(bits, group, block):
    """Section 5 (grouping): a group's grid is fixed when its first column is reached, from the
    weights as the error feedback of all earlier columns has left them -- not from the original
    weights.  By the trajectory identity W0 - W^ = E U (pinned above), the weights of group
    [j, j+g) at that moment are W0[:, j:j+g] - E[:, :j] U[:j, j:j+g]; the returned scale and
    zero-point must be the min-max grid of THAT slice (endpoints checked by brute force over the
    slice), and on strongly correlated inputs they must differ from the original slice's grid."""
    r = RNG(31)
    R, C, m = 12, 64, 400
    Z = r.normal(size=(m, 8)) @ r.normal(size=(8, C)) + 0.05 * r.normal(size=(m, C))
    Xt = _bf16_bits(Z)
    W = (r.normal(size=(R, C)) * 0.02).astype(np.float16)
    H = O.hessian_accumulate(np.zeros((C, C)), Xt)
    U = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0])
    out = O.quantize_layer(W, U, bits, group, False, block=block)
    W0 = W.astype(np.float64)
    maxq = 2 ** bits - 1
    differs = 0
    for j in range(0, C, group):
        gi = j // group
        cur = W0[:, j:j + group] - out["E"][:, :j] @ U[:j, j:j + group]
        s, z = out["scales"][:, gi], out["zeros"][:, gi]
        for rr in range(R):
            lo = min(min(cur[rr]), 0.0)                  # brute force over the slice
            hi = max(max(cur[rr]), 0.0)
            assert s[rr] == np.float64(np.float32((hi - lo) / maxq)), (j, rr)
            # the integer zero-point puts the grid's lower end within half a step of lo
            assert z[rr] == int(z[rr]) and 0 <= z[rr] <= maxq
            assert abs(s[rr] * (0 - z[rr]) - lo) <= 0.5 * s[rr] * (1 + 1e-9)
            lo0 = min(min(W0[rr, j:j + group]), 0.0)
            hi0 = max(max(W0[rr, j:j + group]), 0.0)
            if j > 0 and np.float32((hi0 - lo0) / maxq) != np.float32(s[rr]):
                differs += 1
    # the feedback moves the weights by a good fraction of a step here, so nearly every later
    # group's range differs from the original slice's: a solver that took the grids from W0 fails
    assert differs >= 0.9 * R * (C // group - 1)


# ------------------------------------------------------------------ fp16 scale storage (Section 5, Extreme Quantization)
@pytest.mark.parametrize("bits,group", [(4, 0), (3, 16), (2, 32), (O.BITS_TERNARY, 8)])
def test_fp16_scale_option(bits, group):
    """Section 5 counts one FP16 scale per group in the stored model.  With scale_fp16 the grid is built on the
    fp16-rounded scale: the returned scale is the fp16 value nearest to the unrounded one, the zero-point is derived
    from THAT scale, every code is the nearest level of THAT grid (diagonal H: no feedback, so codes are plain
    nearest-level choices), and scale * (code - zero) needs no rounding in fp32, so the fp16-scale model
    dequantizes to exactly the values the solver compensated for."""
    r = RNG(41)
    R, C = 16, 64
    W = (r.normal(size=(R, C)) * 0.02).astype(np.float16)
    Wd = W.astype(np.float64)
    g = group if group > 0 else C
    maxq = O.maxq_of(bits)
    U = O.cholesky_inverse_upper(np.diag(np.exp(r.normal(size=C))))
    out = O.quantize_layer(W, U, bits, group, False, block=16, scale_fp16=True)
    plain = O.quantize_layer(W, U, bits, group, False, block=16)
    s16 = out["scales"]
    assert np.array_equal(s16, s16.astype(np.float16).astype(np.float64))          # fp16-representable
    if bits != O.BITS_TERNARY:        # (a ternary scale is max|w| of fp16 weights: already an fp16 value)
        assert not np.array_equal(s16, plain["scales"])                            # and it did change something
    for gi in range(C // g):
        seg = Wd[:, gi * g:(gi + 1) * g]
        lo, hi = np.minimum(seg.min(1), 0), np.maximum(seg.max(1), 0)
        exact = (2 * np.maximum(-lo, hi) if bits == O.BITS_TERNARY else (hi - lo)) / maxq
        for rr in range(R):
            s = np.float16(s16[rr, gi])
            for nb in (np.nextafter(s, np.float16(0)), np.nextafter(s, np.float16(np.inf))):
                assert abs(float(s) - exact[rr]) <= abs(float(nb) - exact[rr]) * (1 + 1e-7)   # nearest fp16 value
            z = out["zeros"][rr, gi]
            if bits != O.BITS_TERNARY:
                assert z == np.rint(-lo[rr] / float(s))                            # zero-point from the ROUNDED scale
            for c in range(gi * g, (gi + 1) * g):
                d = np.abs(np.array(_grid_values(float(s), z, maxq)) - Wd[rr, c])
                assert d[out["codes"][rr, c]] == d.min()
    prod32 = (np.repeat(s16, g, 1).astype(np.float32) * (out["codes"] - np.repeat(out["zeros"], g, 1)).astype(np.float32))
    assert np.array_equal(prod32.astype(np.float64), out["W_hat"])                 # exact in fp32
    assert np.array_equal(O.rtn(W, bits, group, False, scale_fp16=True)[0], out["codes"])


# ------------------------------------------------------------------ P8: packed layout
def _golden_pack_vectors():
    path = os.path.join(os.path.dirname(__file__), "golden", "pack_vectors.txt")
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        b, codes, words = [p.strip() for p in line.split(";")]
        yield int(b), np.array([int(c) for c in codes.split()], dtype=np.int32)[None, :], \
            np.array([int(w, 16) for w in words.split()], dtype=np.uint32)[None, :]


def test_pack_golden_vectors():
    n = 0
    for bits, codes, words in _golden_pack_vectors():
        assert np.array_equal(O.pack_codes(codes, bits), words), (bits, codes)
        assert np.array_equal(O.unpack_codes(words, bits, 32), codes)
        n += 1
    assert n >= 6


@pytest.mark.parametrize("bits", [2, 3, 4, 8, O.BITS_TERNARY])
def test_pack_unpack_roundtrip(bits):
    r = RNG(10)
    codes = r.integers(0, O.maxq_of(bits) + 1, size=(7, 96)).astype(np.int32)
    words = O.pack_codes(codes, bits)
    assert words.shape == (7, 96 * O.field_bits_of(bits) // 32) and words.dtype == np.uint32
    assert np.array_equal(O.unpack_codes(words, bits, 96), codes)


# ------------------------------------------------------------------ P9: exact invariances
def test_power_of_two_scaling_invariance_and_on_grid_input():
    W, Xt = _random_problem(8, 64, 300, 11)
    H = O.hessian_accumulate(np.zeros((64, 64)), Xt)
    U = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0])
    a = O.quantize_layer(W, U, 4, 0, False, 32)
    # H -> 4 H: U -> U / 2 exactly; codes unchanged, loss x 4
    b = O.quantize_layer(W, U / 2.0, 4, 0, False, 32)
    assert np.array_equal(a["codes"], b["codes"]) and b["loss"] == pytest.approx(4 * a["loss"], rel=1e-12)
    # W -> 2 W (exact in fp16): codes unchanged, scales doubled
    c = O.quantize_layer((W * np.float16(2)).astype(np.float16), U, 4, 0, False, 32)
    assert np.array_equal(a["codes"], c["codes"]) and np.array_equal(c["scales"], 2 * a["scales"])
    # a W that already lies on its own grid is reproduced with zero loss
    lv = RNG(12).integers(0, 16, size=(8, 64))
    lv[:, 0], lv[:, 1] = 0, 15
    Wg = ((lv - 8) * 2.0 ** -7).astype(np.float16)
    d = O.quantize_layer(Wg, U, 4, 0, False, 32)
    assert np.array_equal(d["codes"], lv) and d["loss"] == 0.0
    assert np.array_equal(d["W_hat"], Wg.astype(np.float64))


def test_rows_are_independent():
    """Eq. 1 splits over rows (Section 2): solving a subset of rows gives the same rows."""
    W, Xt = _random_problem(12, 64, 300, 13)
    H = O.hessian_accumulate(np.zeros((64, 64)), Xt)
    U = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0])
    full = O.quantize_layer(W, U, 3, 32, False, 32)
    part = O.quantize_layer(W[[2, 5, 11]], U, 3, 32, False, 32)
    assert np.array_equal(full["codes"][[2, 5, 11]], part["codes"])
    assert np.array_equal(full["scales"][[2, 5, 11]], part["scales"])


# ------------------------------------------------------------------ dequantize / matvec (Section 5, Practical Speedups)
def test_dequantize_and_matvec_definitions():
    r = RNG(15)
    W = (r.normal(size=(6, 64)) * 0.02).astype(np.float16)
    U = np.eye(64)
    out = O.quantize_layer(W, U, 3, 32, False, 32)
    deq = O.dequantize(out["codes"], out["scales"], out["zeros"])
    assert np.array_equal(deq, out["W_hat"])                    # the same grid points the solver produced
    # hand check of one entry, and a level-by-level brute force of the whole matrix
    s, z, q = out["scales"][2, 1], out["zeros"][2, 1], out["codes"][2, 40]
    assert deq[2, 40] == s * (q - z)
    x = (r.normal(size=64)).astype(np.float16)
    y = O.matvec(out["codes"], out["scales"], out["zeros"], x)
    want = [sum(float(deq[i, c]) * float(x[c]) for c in range(64)) for i in range(6)]
    assert np.allclose(y, want, rtol=1e-12)
    # fp16 storage reading: within half an fp16 ulp of the exact value
    d16 = O.dequantize(out["codes"], out["scales"], out["zeros"], to_fp16=True)
    assert d16.dtype == np.float16 and np.all(np.abs(d16.astype(np.float64) - deq) <= np.abs(deq) * 2.0 ** -11 + 1e-12)


@pytest.mark.parametrize("bits,group", [(4, 0), (3, 16), (2, 0)])
def test_residuals_through_the_factor_give_the_lazy_update(bits, group):
    """The identity the CUDA path's factor form rests on, checked on the oracle's own trajectory.  Algorithm 1's updates
    sum to W - Q = E U; hence E = (W - Q) U~ with U~ = U^-1 (the upper factor of the damped Hessian, H~ = U~ U~^T), and for
    any block J of columns, what the lazy updates have subtracted from block J when the loop reaches it,
    E[:, :j0] U[:j0, J], equals -((W - Q)[:, :j0] U~[:j0, J]) U[J, J]."""
    C, blk = 96, 32
    W, Xt = _random_problem(12, C, 400, 21)
    H = O.hessian_accumulate(np.zeros((C, C)), Xt)
    Ht, _ = O.dampen(H, 0.01)
    U = O.cholesky_inverse_upper(Ht)
    Ut = np.linalg.inv(U)
    assert np.allclose(Ut @ Ut.T, Ht, rtol=1e-10, atol=1e-12 * np.abs(Ht).max())          # U~ is the factor of H~ itself
    out = O.quantize_layer(W, U, bits, group, False, block=16)
    Rm = W.astype(np.float64) - out["W_hat"]                                               # plain residuals w - q
    assert np.allclose(out["E"], Rm @ Ut, rtol=1e-8, atol=1e-12)
    for j0 in range(blk, C, blk):
        J = slice(j0, j0 + blk)
        lazy = out["E"][:, :j0] @ U[:j0, J]
        through_factor = -(Rm[:, :j0] @ Ut[:j0, J]) @ U[J, J]
        assert np.allclose(lazy, through_factor, rtol=1e-8, atol=1e-12)


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_symmetric_grid_puts_minus_max_on_a_tie(bits):
    """The symmetric option (not defined by the paper): scale = 2a / maxq and zero = (maxq + 1) / 2 with an even number of
    levels put -a exactly midway between codes 0 and 1, so in real arithmetic both are nearest; which one the oracle
    returns follows the fp32 rounding of the scale.  Over many values of a both codes occur, the chosen grid value is
    always one of the two nearest, and +a (which maps past the top level) always clamps to maxq.  This is why GPU parity
    for symmetric grids compares rows only up to the first such tie."""
    maxq = O.maxq_of(bits)
    r = np.random.default_rng(bits)
    a = np.exp(r.normal(size=4000)).astype(np.float16).astype(np.float64)
    lo = np.stack([-a, 0.25 * a], 1)                         # the row's largest magnitude is negative
    scale, zero = O.find_params(lo, bits, True)
    assert np.array_equal(zero, np.full_like(zero, (maxq + 1) // 2))
    assert np.array_equal(scale, (2.0 * a / maxq).astype(np.float32).astype(np.float64))
    q, wq = O.quant(lo[:, 0], scale, zero, maxq)
    assert set(np.unique(q)) == {0.0, 1.0}                   # both sides of the tie occur
    exact = -a / (2.0 * a / maxq) + (maxq + 1) // 2          # position of -a on the exact grid
    assert np.allclose(exact, 0.5)
    d0, d1 = np.abs(lo[:, 0] - scale * (0 - zero)), np.abs(lo[:, 0] - scale * (1 - zero))
    assert np.all(np.abs(d0 - d1) <= 1e-6 * a)               # equally near up to the scale's rounding
    assert np.all(np.abs(lo[:, 0] - wq) <= np.minimum(d0, d1) + 1e-12)
    hi = np.stack([a, -0.25 * a], 1)                         # largest magnitude positive: past the top level, clamped
    scale, zero = O.find_params(hi, bits, True)
    assert np.array_equal(O.quant(hi[:, 0], scale, zero, maxq)[0], np.full(len(a), float(maxq)))

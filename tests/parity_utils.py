"""Comparison helpers for the GPU-vs-oracle parity tests (tolerances of the benchmark spec)."""
import numpy as np

from oracle import gptq_oracle as O

TOL_H_FRO = 1e-5          # relative Frobenius error of H
TOL_CODES_IDENTICAL = 0.999   # fraction of identical integer codes; every mismatch exactly +-1 level
TOL_SCALE_ZERO = 1e-5     # relative error of scales and zeros
TOL_RECON = 0.01          # relative difference of ||W X - W^ X||_F^2
TOL_U_FRO = 2e-5          # fp32 factorisation of a matrix with relative diagonal range ~1e6


def rel_fro(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def check_quantize_outputs(gpu, ref, W16, bits, C, H=None, min_identical=TOL_CODES_IDENTICAL):
    """gpu: dict of numpy arrays from the CUDA path (qweight uint32, scales, zeros, loss).
    ref: oracle quantize_layer dict.  Returns a dict of measured figures."""
    qw = gpu["qweight"].view(np.uint32)
    codes = O.unpack_codes(qw, bits, C)
    # packed layout: bit-exact against the oracle's packer applied to the same codes
    assert np.array_equal(O.pack_codes(codes, bits), qw), "packed layout differs"
    assert codes.min() >= 0 and codes.max() <= O.maxq_of(bits)
    diff = codes - ref["codes"]
    identical = float((diff == 0).mean())
    assert np.abs(diff).max() <= 1, f"a code differs by more than one level (max {np.abs(diff).max()})"
    assert identical >= min_identical, f"only {identical:.5f} of the codes identical"
    s_err = rel_fro(gpu["scales"], ref["scales"])
    z_err = rel_fro(gpu["zeros"], ref["zeros"])
    assert s_err <= TOL_SCALE_ZERO, f"scales rel err {s_err}"
    assert z_err <= TOL_SCALE_ZERO, f"zeros rel err {z_err}"
    out = dict(identical=identical, scales_err=s_err, zeros_err=z_err)
    g = C // gpu["scales"].shape[1]
    What = gpu["scales"].astype(np.float64).repeat(g, 1) * (codes - gpu["zeros"].astype(np.float64).repeat(g, 1))
    if H is not None:
        r_gpu = O.reconstruction_error(W16, What, H)
        r_ref = O.reconstruction_error(W16, ref["W_hat"], H)
        assert abs(r_gpu - r_ref) <= TOL_RECON * r_ref, f"reconstruction loss {r_gpu} vs {r_ref}"
        out["recon_ratio"] = r_gpu / r_ref
    loss = float(gpu["loss"])
    assert abs(loss - ref["loss"]) <= TOL_RECON * ref["loss"] + 1e-30, f"loss {loss} vs {ref['loss']}"
    out["loss_ratio"] = loss / ref["loss"] if ref["loss"] else 1.0
    return out

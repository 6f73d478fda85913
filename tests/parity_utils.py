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


def check_quantize_outputs(gpu, ref, W16, bits, C, H=None, min_identical=TOL_CODES_IDENTICAL, scale_fp16=False):
    """gpu: dict of numpy arrays from the CUDA path (qweight uint32, scales, zeros, loss).
    ref: oracle quantize_layer dict.  Returns a dict of measured figures.
    scale_fp16: the scales are fp16 values, each a rounding decision taken from working weights that the two sides hold
    to about 1e-7 of each other, so a scale next to an fp16 rounding boundary may fall on either side of it; the row then
    continues on another grid.  Such rows (rare) are left out of the code comparison; loss and reconstruction are still
    compared over all rows."""
    qw = gpu["qweight"].view(np.uint32)
    codes = O.unpack_codes(qw, bits, C)
    # packed layout: bit-exact against the oracle's packer applied to the same codes
    assert np.array_equal(O.pack_codes(codes, bits), qw), "packed layout differs"
    assert codes.min() >= 0 and codes.max() <= O.maxq_of(bits)
    rows = np.ones(codes.shape[0], dtype=bool)          # rows whose grids are the oracle's
    s_err = rel_fro(gpu["scales"], ref["scales"])
    z_err = rel_fro(gpu["zeros"], ref["zeros"])
    if scale_fp16:
        hg = gpu["scales"].astype(np.float16)
        hr = ref["scales"].astype(np.float16)
        assert np.array_equal(hg.astype(np.float32), gpu["scales"].astype(np.float32)), "a scale is not an fp16 value"
        ulps = np.abs(hg.view(np.int16).astype(np.int32) - hr.view(np.int16).astype(np.int32))
        # a row in which a scale fell on the other side of an fp16 rounding boundary has another grid from there on: its
        # codes are not compared; such rows must stay rare, and their scales at most one fp16 unit away where they first differ
        rows = (ulps == 0).all(axis=1)
        assert rows.mean() >= 0.95, f"only {rows.mean():.3f} of the rows have the oracle's fp16 scales"
        for r in np.where(~rows)[0]:
            assert ulps[r, int(np.argmax(ulps[r] > 0))] == 1, f"row {r}: first differing scale is more than one fp16 unit away"
    else:
        assert s_err <= TOL_SCALE_ZERO, f"scales rel err {s_err}"
    diff = (codes - ref["codes"])[rows]
    identical = float((diff == 0).mean())
    assert np.abs(diff).max() <= 1, f"a code differs by more than one level (max {np.abs(diff).max()})"
    assert identical >= min_identical, f"only {identical:.5f} of the codes identical"
    z_rows = rel_fro(gpu["zeros"][rows], ref["zeros"][rows])
    assert z_rows <= TOL_SCALE_ZERO, f"zeros rel err {z_rows}"
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


# ---- checks that work at any size (H and U are CUDA tensors; torch is imported lazily) -----------------
def check_hessian_sampled(L, H, n_cols=24):
    """Sampled entries of H against the definition 2 sum_t x_ti x_tj, from host-generated columns of X."""
    import torch
    r = np.random.default_rng(5 + L.C)
    cols = np.unique(np.concatenate([r.integers(0, L.C, n_cols), [0, L.C - 1, 127, 128, 255, 256]]))
    sc = L.scales()
    Xc = np.concatenate([O.bf16_bits_to_f64(L.x_bits(t0, min(t0 + 32768, L.n_tokens), cols=cols, scales=sc))
                         for t0 in range(0, L.n_tokens, 32768)])
    ref = 2.0 * (Xc.T @ Xc)
    idx = torch.from_numpy(cols).cuda()
    got = H[idx][:, idx].cpu().numpy().astype(np.float64)
    fro = float(np.linalg.norm(got - ref) / np.linalg.norm(ref))
    assert fro <= TOL_H_FRO, fro
    assert np.abs(got - ref).max() <= 1e-5 * np.abs(ref).max()
    d = np.diag(ref)
    assert (np.abs(np.diag(got) - d) <= 5e-6 * d).all()
    return fro


def check_factor_on_device(H, U, damp, k_tail=512, n_probe=4, blk=2048):
    """U upper with positive diagonal; probe residual of U^T U = (H + lambda I)^-1 in fp64 (device, row blocks);
    last rows of U against the oracle's literal route on the trailing principal block of H~."""
    import torch
    C = H.shape[0]
    assert bool((torch.diagonal(U) > 0).all())
    for r0 in range(0, C, blk):                              # strict lower triangle is exactly zero
        r1 = min(C, r0 + blk)
        assert not bool(torch.tril(U[r0:r1, :r1], diagonal=r0 - 1).any()), r0
    lam = damp * float(torch.diagonal(H).double().mean().item())
    g = torch.Generator(device="cuda").manual_seed(6)
    z = torch.randn((C, n_probe), dtype=torch.float64, device="cuda", generator=g)
    y = torch.empty_like(z)
    for r0 in range(0, C, blk):
        y[r0:r0 + blk] = U[r0:r0 + blk].double() @ z
    w = torch.zeros_like(z)
    for r0 in range(0, C, blk):
        w += U[r0:r0 + blk].double().T @ y[r0:r0 + blk]
    v = lam * w
    for r0 in range(0, C, blk):
        v[r0:r0 + blk] += H[r0:r0 + blk].double() @ w
    res = float(((v - z).norm(dim=0) / z.norm(dim=0)).max().item())
    assert res <= 5e-5, res
    Ht_tail = H[C - k_tail:, C - k_tail:].cpu().numpy().astype(np.float64)
    Ht_tail[np.diag_indices_from(Ht_tail)] += lam
    Uref = O.cholesky_inverse_upper(Ht_tail)
    Ut = U[C - k_tail:, C - k_tail:].cpu().numpy().astype(np.float64)
    err = float((np.linalg.norm(Ut - Uref, axis=1) / np.linalg.norm(Uref, axis=1)).max())
    assert err <= 1e-4, err
    return res, err

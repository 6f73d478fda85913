"""Parity on every workload BASELINE names, at full calibration size (262144 tokens), through the three C-ABI
calls exactly as bench.py issues them.

  config 1  one whole OPT-125M-shaped block (six layers x {4-bit, 3-bit} per row): the oracle solves every layer
            END TO END (its own H, its own U) and the GPU's H -> U -> codes are compared with that.
  config 2  'q' (4096 x 4096), 3-bit g128: end to end against the oracle's own H and U on sampled rows.
  config 3  'q' (12288 x 12288) and 'fc2' (12288 x 49152), 4-bit and 3-bit per row: stage by stage, on what the
            oracle can compute one by one (sampled entries of H from host-generated columns, probe residual and
            trailing-block factor for U, sampled rows of stage 3 re-solved by the oracle with the GPU's U).
  config 4  'fc2' (14336 x 57344), 2-bit g128 and ternary g128: the same stage-by-stage scheme.

The probe residual || H~ U^T (U z) - z || / || z || is a property check, not an oracle value; at these sizes it is
evaluated in fp64 with torch on the device (row blocks of H and U promoted to double), which is test arithmetic only.
Activations of the big layers come from the device filler, whose output is bit-identical to the host generator
(checked here again on sampled token ranges before the oracle is fed with it).
"""
import json
import os
import time

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import gptq_oracle as O
from paper_2210_17323_b200.synth import workloads as WL
from tests.parity_utils import (TOL_H_FRO, TOL_U_FRO, check_factor_on_device, check_hessian_sampled,
                                check_quantize_outputs, rel_fro)

FIGURES = {}      # measured parity figures per case, printed at the end of the module (pytest -s shows them)


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_17323_b200 import binding
    return binding


@pytest.fixture(scope="module")
def D():
    from paper_2210_17323_b200.synth import device
    return device


def _x_to_host_checked(L, X):
    """Device-filled activations as host bf16 bit patterns, after re-checking sampled token ranges against the
    host generator (the oracle's inputs are the seeded generator's, whichever side produced the bytes)."""
    bits = X.view(torch.int16).cpu().numpy().view(np.uint16)
    r = np.random.default_rng(L.C + L.R)
    for t0 in [0, L.n_tokens - 64] + list(r.integers(0, L.n_tokens - 64, 3)):
        t0 = int(t0)
        assert np.array_equal(bits[t0:t0 + 64], L.x_bits(t0, t0 + 64)), (L.name, t0)
    return bits


def _solve_gpu(B, D, L, wl, grids, keep_x=False):
    X = D.fill_x(L)
    W = D.fill_w(L)
    H = torch.zeros((L.C, L.C), dtype=torch.float32, device="cuda")
    info_h = torch.zeros(2, dtype=torch.int32, device="cuda")
    B.gptq_hessian_accumulate(H, X, dev_info=info_h)
    if not keep_x:
        del X
    U, info = B.gptq_prepare_hinv(H, wl.damp)
    outs = []
    for g in grids:
        o = B.gptq_quantize_layer(W, U, g.bits, g.group_size, g.sym, wl.block)
        outs.append(o)
    # the same layer in the factor form (stage 2 without the inverse, stage 3 on the factor)
    F, info_f = B.gptq_prepare_hinv(H, wl.damp, factor=True)
    outs_f = [B.gptq_quantize_layer(W, F, g.bits, g.group_size, g.sym, wl.block, factor=True) for g in grids]
    torch.cuda.synchronize()
    assert info_h.tolist()[0] == 0 and info.tolist()[0] == 0 and info_f.tolist()[0] == 0
    assert all(o["dev_info"].tolist()[0] == 0 for o in outs + outs_f)
    _check_factor_against_u(F, U)
    del F
    return dict(H=H, U=U, outs=outs, outs_factor=outs_f, X=X if keep_x else None)


def _check_factor_against_u(F, U, blk=1024):
    """gptq_prepare_factor's output against gptq_prepare_hinv's on the device: the same diagonal blocks up to rounding, and for the last
    block of columns J the identity U[:j0, J] = -U[:j0, :j0] F[:j0, J] (F[:j0, J] = U~[:j0, J] U_JJ) on a probe vector, in
    fp64 row chunks."""
    C = U.shape[0]
    for j0 in range(0, C, blk):
        j1 = min(C, j0 + blk)
        d = (F[j0:j1, j0:j1].double() - U[j0:j1, j0:j1].double()).norm() / U[j0:j1, j0:j1].double().norm()
        assert d.item() <= 1e-5, (j0, d.item())      # (two runs of the factorisation: their reductions add in different orders)
    j0 = (C - 1) // blk * blk
    if j0 == 0:
        return
    g = torch.Generator(device="cuda").manual_seed(5)
    z = torch.randn(C - j0, dtype=torch.float64, device="cuda", generator=g)
    v = F[:j0, j0:].double() @ z
    lhs = U[:j0, j0:].double() @ z
    rhs = torch.empty_like(lhs)
    for r0 in range(0, j0, 4096):
        r1 = min(j0, r0 + 4096)
        rhs[r0:r1] = -(U[r0:r1, :j0].double() @ v)
    err = ((lhs - rhs).norm() / lhs.norm()).item()
    assert err <= 1e-4, err


def _gpu_out_rows(o, rows=None):
    sl = slice(None) if rows is None else torch.from_numpy(np.asarray(rows)).cuda()
    return dict(qweight=o["qweight"][sl].cpu().numpy(), scales=o["scales"][sl].cpu().numpy(),
                zeros=o["zeros"][sl].cpu().numpy(), loss=o["loss"].item())


def _check_rows(L, wl, g, U64, o, n_rows, H64=None, seed=7, o_factor=None):
    """Rows are independent sub-problems (Section 2): a sample of them, re-solved by the oracle with the GPU's U.
    o_factor: the factor form's outputs for the same layer, checked against the same oracle result."""
    rows = np.sort(np.random.default_rng(seed + L.R).choice(L.R, n_rows, replace=False))
    W16 = L.w(rows=rows)
    ref = O.quantize_layer(W16, U64, g.bits, g.group_size, g.sym, wl.block)
    per_row = ref["loss"] / n_rows
    figs = None
    for out in (o_factor, o):                  # (the figures reported are the last one's: the form Algorithm 1 writes)
        if out is None:
            continue
        gpu = _gpu_out_rows(out, rows)
        layer_loss = gpu["loss"]
        gpu["loss"] = ref["loss"]              # the layer's loss covers all rows: checked below on the sample's share
        f = check_quantize_outputs(gpu, ref, W16, g.bits, L.C, H64)
        assert 0.5 * per_row * L.R <= layer_loss <= 2.0 * per_row * L.R
        if out is o_factor:
            figs_factor = f
        figs = f
    if o_factor is not None:
        figs["identical_factor_form"] = figs_factor["identical"]
    figs["rows"] = int(n_rows)
    return figs


# ------------------------------------------------------------------ config 1: one block, every layer end to end
def test_config1_block_end_to_end(B, D):
    wl = WL.workload(1)
    block0 = [l for l in wl.layers if l.block_idx == 0]
    assert [l.kind for l in block0] == ["q", "k", "v", "o", "fc1", "fc2"]
    for L in block0:
        t0 = time.time()
        s = _solve_gpu(B, D, L, wl, wl.grids, keep_x=True)
        bits = _x_to_host_checked(L, s["X"])
        s["X"] = None
        W16 = L.w()
        H = O.hessian_accumulate(np.zeros((L.C, L.C)), bits, chunk=16384)
        Ht, _ = O.dampen(H, wl.damp)
        U = O.cholesky_inverse_upper(Ht)
        h_err = rel_fro(s["H"].cpu().numpy(), H)
        u_err = rel_fro(s["U"].cpu().numpy(), U)
        assert h_err <= TOL_H_FRO and u_err <= TOL_U_FRO, (L.name, h_err, u_err)
        for g, o, of in zip(wl.grids, s["outs"], s["outs_factor"]):
            ref = O.quantize_layer(W16, U, g.bits, g.group_size, g.sym, wl.block)
            figs_f = check_quantize_outputs(_gpu_out_rows(of), ref, W16, g.bits, L.C, H)      # the factor form
            figs = check_quantize_outputs(_gpu_out_rows(o), ref, W16, g.bits, L.C, H)
            figs["identical_factor_form"] = figs_f["identical"]
            figs.update(H_rel_fro=h_err, U_rel_fro=u_err, seconds=round(time.time() - t0, 1))
            FIGURES[f"c1 {L.kind} {L.R}x{L.C} bits={g.bits} end-to-end"] = figs


# ------------------------------------------------------------------ config 2: q layer end to end
def test_config2_q_end_to_end_sampled_rows(B, D):
    wl = WL.workload(2)
    L = [l for l in wl.layers if l.kind == "q"][0]
    g = wl.grids[0]
    s = _solve_gpu(B, D, L, wl, wl.grids, keep_x=True)
    bits = _x_to_host_checked(L, s["X"])
    s["X"] = None
    H = O.hessian_accumulate(np.zeros((L.C, L.C)), bits, chunk=16384)
    del bits
    U = O.cholesky_inverse_upper(O.dampen(H, wl.damp)[0])
    h_err = rel_fro(s["H"].cpu().numpy(), H)
    u_err = rel_fro(s["U"].cpu().numpy(), U)
    assert h_err <= TOL_H_FRO and u_err <= TOL_U_FRO, (h_err, u_err)
    figs = _check_rows(L, wl, g, U, s["outs"][0], 64, H, o_factor=s["outs_factor"][0])   # the ORACLE's U: end-to-end comparison
    figs.update(H_rel_fro=h_err, U_rel_fro=u_err)
    FIGURES[f"c2 q {L.R}x{L.C} bits={g.bits} g{g.group_size} end-to-end (64 rows)"] = figs


# ------------------------------------------------------------------ configs 3 and 4: stage by stage
def _stagewise(B, D, cfg, kind, n_rows):
    wl = WL.workload(cfg)
    L = [l for l in wl.layers if l.kind == kind][0]
    s = _solve_gpu(B, D, L, wl, wl.grids)
    h_fro = check_hessian_sampled(L, s["H"])
    res, tail = check_factor_on_device(s["H"], s["U"], wl.damp)
    U64 = s["U"].cpu().numpy().astype(np.float64)
    s["H"] = None
    for g, o, of in zip(wl.grids, s["outs"], s["outs_factor"]):
        figs = _check_rows(L, wl, g, U64, o, n_rows, o_factor=of)
        figs.update(H_sampled_rel_fro=h_fro, U_probe_residual=res, U_tail_rows_err=tail)
        FIGURES[f"c{cfg} {kind} {L.R}x{L.C} bits={g.bits} g{g.group_size} stage-isolated"] = figs


def test_config3_q_stagewise(B, D):
    _stagewise(B, D, 3, "q", 24)


def test_config3_fc2_stagewise(B, D):
    _stagewise(B, D, 3, "fc2", 12)


def test_config4_fc2_stagewise(B, D):
    _stagewise(B, D, 4, "fc2", 12)


def test_zz_report_figures():
    """Prints the measured figures of this module; also written as JSON to $GPTQ_PARITY_REPORT when that is set."""
    for k, v in FIGURES.items():
        print(k, {a: (round(b, 8) if isinstance(b, float) else b) for a, b in v.items()})
    path = os.environ.get("GPTQ_PARITY_REPORT")
    if path:
        with open(path, "w") as f:
            json.dump(FIGURES, f, indent=1)

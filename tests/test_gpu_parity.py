"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle, element by element."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import gptq_oracle as O
from paper_2210_17323_b200.synth import generator as G, workloads as WL
from tests.parity_utils import (TOL_H_FRO, TOL_U_FRO, check_quantize_outputs, rel_fro)


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


def _np_bf16_to_torch(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _layer(R, C, m, cfg=9, blk=0, kind="q"):
    return WL.Layer(cfg, blk, kind, R, C, m)


def _run_quant(B, W16, U32, bits, group, sym, block):
    out = B.gptq_quantize_layer(torch.from_numpy(W16).cuda(), torch.from_numpy(U32).cuda(), bits, group, sym, block)
    torch.cuda.synchronize()
    assert out["dev_info"].tolist()[0] == 0
    return dict(qweight=out["qweight"].cpu().numpy(), scales=out["scales"].cpu().numpy(),
                zeros=out["zeros"].cpu().numpy(), loss=out["loss"].item())


# ------------------------------------------------------------------ inputs
def test_device_filler_matches_host_generator(D):
    L = _layer(96, 160, 300)
    X = D.fill_x(L).view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(X, L.x_bits())
    assert np.array_equal(D.fill_x(L, 17, 200).view(torch.int16).cpu().numpy().view(np.uint16), L.x_bits(17, 200))
    W = D.fill_w(L).cpu().numpy()
    assert np.array_equal(W.view(np.uint16), L.w().view(np.uint16))


# ------------------------------------------------------------------ stage 1
@pytest.mark.parametrize("C,m", [(32, 1), (96, 77), (160, 1000), (256, 4096), (768, 8192), (1056, 777), (544, 1)])
def test_hessian_matches_oracle(B, C, m):
    L = _layer(8, C, m)
    bits = L.x_bits()
    H = torch.zeros((C, C), dtype=torch.float32, device="cuda")
    B.gptq_hessian_accumulate(H, _np_bf16_to_torch(bits))
    Hg = H.cpu().numpy()
    Href = O.hessian_accumulate(np.zeros((C, C)), bits)
    assert rel_fro(Hg, Href) <= TOL_H_FRO
    assert np.array_equal(Hg, Hg.T)


def test_hessian_integer_inputs_bit_exact_and_chunked(B):
    r = np.random.default_rng(3)
    C, m = 160, 700
    Xi = r.integers(-8, 9, size=(m, C)).astype(np.float32)
    Xt = torch.from_numpy(Xi).cuda().to(torch.bfloat16)
    H = torch.zeros((C, C), dtype=torch.float32, device="cuda")
    for a, b in ((0, 33), (33, 512), (512, 700)):      # accumulate over ragged chunks
        B.gptq_hessian_accumulate(H, Xt[a:b].contiguous())
    exact = 2.0 * (Xi.astype(np.float64).T @ Xi.astype(np.float64))
    assert np.array_equal(H.cpu().numpy().astype(np.float64), exact)
    B.gptq_hessian_accumulate(H, Xt[:0].contiguous())   # empty batch: no-op
    assert np.array_equal(H.cpu().numpy().astype(np.float64), exact)


@pytest.mark.parametrize("C", [160, 1056])
def test_hessian_chunks_into_the_upper_triangle_then_one_mirror(B, C):
    """gptq_hessian_accumulate_upper adds to the upper triangle only and never writes strictly below the diagonal tiles'
    rows; the last chunk (gptq_hessian_accumulate) or gptq_hessian_symmetrize completes H.  Integer-valued inputs: every
    result is exact, so the chunked sum must equal the one-call sum bit for bit."""
    r = np.random.default_rng(C)
    m = 900
    Xi = r.integers(-8, 9, size=(m, C)).astype(np.float32)
    Xt = torch.from_numpy(Xi).cuda().to(torch.bfloat16)
    exact = 2.0 * (Xi.astype(np.float64).T @ Xi.astype(np.float64))
    H = torch.zeros((C, C), dtype=torch.float32, device="cuda")
    B.gptq_hessian_accumulate(H, Xt[:100].contiguous(), upper_only=True)
    B.gptq_hessian_accumulate(H, Xt[100:577].contiguous(), upper_only=True)
    Hu = H.cpu().numpy().astype(np.float64)
    part = 2.0 * (Xi[:577].astype(np.float64).T @ Xi[:577].astype(np.float64))
    assert np.array_equal(np.triu(Hu), np.triu(part))                     # the upper triangle is complete after every call
    B.gptq_hessian_accumulate(H, Xt[577:].contiguous())                     # the last chunk mirrors
    assert np.array_equal(H.cpu().numpy().astype(np.float64), exact)
    H2 = torch.zeros((C, C), dtype=torch.float32, device="cuda")
    B.gptq_hessian_accumulate(H2, Xt, upper_only=True)
    B.gptq_hessian_symmetrize(H2)
    assert np.array_equal(H2.cpu().numpy().astype(np.float64), exact)


# ------------------------------------------------------------------ stage 2
@pytest.mark.parametrize("C", [32, 96, 160, 768, 1056, 2304])
def test_prepare_hinv_matches_oracle(B, C):
    L = _layer(8, C, 2 * C + 100)
    H64 = O.hessian_accumulate(np.zeros((C, C)), L.x_bits())
    H32 = H64.astype(np.float32)
    U, info = B.gptq_prepare_hinv(torch.from_numpy(H32).cuda(), 0.01)
    torch.cuda.synchronize()
    assert info.tolist() == [0, 0]
    Ug = U.cpu().numpy()
    Uref = O.cholesky_inverse_upper(O.dampen(H32.astype(np.float64), 0.01)[0])
    assert np.array_equal(Ug, np.triu(Ug)) and (np.diag(Ug) > 0).all()
    assert rel_fro(Ug, Uref) <= TOL_U_FRO
    # row-wise: every row of U from the diagonal on, relative to that row's norm
    row_err = np.linalg.norm(Ug - Uref, axis=1) / np.linalg.norm(Uref, axis=1)
    assert row_err.max() <= 1e-4


def test_prepare_hinv_reports_not_positive_definite(B):
    C = 64
    H = np.eye(C, dtype=np.float32)
    H[10, 20] = H[20, 10] = 5.0      # indefinite
    U, info = B.gptq_prepare_hinv(torch.from_numpy(H).cuda(), 0.01)
    torch.cuda.synchronize()
    st, where = info.tolist()
    assert st == B.ERR_NOT_PD and 0 <= where < C
    assert torch.isfinite(U).all()
    # all-zero H (no calibration data): damping cannot help
    U, info = B.gptq_prepare_hinv(torch.zeros((C, C), device="cuda"), 0.01)
    torch.cuda.synchronize()
    assert info.tolist()[0] == B.ERR_NOT_PD


# ------------------------------------------------------------------ stage 3 (oracle's U on both sides)
CASES = [
    # R,   C,   bits, group, sym, block
    (200, 768, 4, 0, False, 128),
    (129, 160, 3, 0, False, 128),      # ragged rows, short last block
    (7, 96, 4, 0, False, 32),
    (1, 32, 2, 0, False, 32),
    (300, 512, 3, 128, False, 128),
    (300, 512, 2, 128, False, 64),     # group wider than block
    (300, 512, 2, 128, False, 256),    # block wider than group
    (64, 256, O.BITS_TERNARY, 128, False, 32),
    (64, 256, 4, 16, False, 128),      # small groups inside the register sub-block
    (64, 256, 8, 0, False, 128),
    (64, 256, 4, 64, True, 64),        # symmetric grid
    (260, 2304, 4, 0, False, 128),     # several outer (lazy) blocks
    (130, 2176, 3, 32, False, 96),     # block that is not a power of two (groups of 32 nest in it); ragged outer block
    (64, 2048, O.BITS_TERNARY, 8, False, 128),   # the paper's ternary setting: group size 8
    (64, 2048, 4, 1024, False, 128),             # group size 1024 (group spans eight blocks)
    (64, 2048, 2, 32, False, 128),               # group size 32
]


@pytest.mark.parametrize("R,C,bits,group,sym,block", CASES)
def test_quantize_layer_matches_oracle(B, R, C, bits, group, sym, block):
    assert not (group and (group % block and block % group)), "cases must have nested group and block sizes"
    L = _layer(R, C, 2 * C + 64, cfg=8)
    W16 = L.w()
    H = O.hessian_accumulate(np.zeros((C, C)), L.x_bits())
    U32 = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0]).astype(np.float32)
    ref = O.quantize_layer(W16, U32.astype(np.float64), bits, group, sym, block)
    gpu = _run_quant(B, W16, U32, bits, group, sym, block)
    check_quantize_outputs(gpu, ref, W16, bits, C, H)


@pytest.mark.parametrize("R,C,bits,group,sym,block", [CASES[0], CASES[1], CASES[4], CASES[5], CASES[8], CASES[11], CASES[12], CASES[14]])
def test_quantize_layer_per_block_form_matches_oracle(B, R, C, bits, group, sym, block):
    """The other form of the loops inside an outer block (one in-block kernel plus one small tensor-core contraction per
    inner block instead of the row-stripe kernel): same parity bar, and its codes agree with the default form's."""
    L = _layer(R, C, 2 * C + 64, cfg=8)
    W16 = L.w()
    H = O.hessian_accumulate(np.zeros((C, C)), L.x_bits())
    U32 = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0]).astype(np.float32)
    ref = O.quantize_layer(W16, U32.astype(np.float64), bits, group, sym, block)
    stripe = _run_quant(B, W16, U32, bits, group, sym, block)
    prev = B.gptq_set_stage3_variant(0)
    try:
        assert prev == 1
        gpu = _run_quant(B, W16, U32, bits, group, sym, block)
    finally:
        B.gptq_set_stage3_variant(prev)
    check_quantize_outputs(gpu, ref, W16, bits, C, H)
    a = O.unpack_codes(gpu["qweight"].view(np.uint32), bits, C)
    b = O.unpack_codes(stripe["qweight"].view(np.uint32), bits, C)
    assert (a == b).mean() >= 0.999


@pytest.mark.parametrize("bits,group,sym", [(4, 0, False), (3, 128, False), (O.BITS_TERNARY, 8, False), (4, 64, True)])
def test_quantize_and_rtn_with_fp16_scales(B, bits, group, sym):
    """Scales rounded to fp16 when the grid is fixed (the stored model's scale precision, Section 5): solver and RTN
    against the oracle run with the same option; returned scales are fp16-representable."""
    R, C = 96, 1024
    L = _layer(R, C, 2 * C + 64, cfg=5)
    W16 = L.w()
    H = O.hessian_accumulate(np.zeros((C, C)), L.x_bits())
    U32 = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0]).astype(np.float32)
    ref = O.quantize_layer(W16, U32.astype(np.float64), bits, group, sym, 128, scale_fp16=True)
    out = B.gptq_quantize_layer(torch.from_numpy(W16).cuda(), torch.from_numpy(U32).cuda(), bits, group, sym, 128, scale_fp16=True)
    torch.cuda.synchronize()
    assert out["dev_info"].tolist()[0] == 0
    gpu = dict(qweight=out["qweight"].cpu().numpy(), scales=out["scales"].cpu().numpy(), zeros=out["zeros"].cpu().numpy(),
               loss=out["loss"].item())
    check_quantize_outputs(gpu, ref, W16, bits, C, H)
    assert np.array_equal(gpu["scales"], gpu["scales"].astype(np.float16).astype(np.float32))
    rt = B.gptq_rtn_layer(torch.from_numpy(W16).cuda(), bits, group, sym, scale_fp16=True)
    codes_ref, _ = O.rtn(W16, bits, group, sym, scale_fp16=True)
    assert np.array_equal(O.unpack_codes(rt["qweight"].cpu().numpy().view(np.uint32), bits, C), codes_ref)
    # flag bits beyond the two defined ones are rejected
    Wd = torch.from_numpy(W16).cuda()
    st = B._lib.gptq_rtn_layer(Wd.data_ptr(), R, C, 4, 0, 4, rt["qweight"].data_ptr(), rt["scales"].data_ptr(),
                               rt["zeros"].data_ptr(), None)
    assert st == B.ERR_INVALID_ARG


def test_prepare_hinv_in_place(B):
    """U may be the same buffer as H: the factor replaces the Hessian."""
    C = 1280
    L = _layer(8, C, 3000, cfg=4)
    H32 = O.hessian_accumulate(np.zeros((C, C)), L.x_bits()).astype(np.float32)
    Uref = O.cholesky_inverse_upper(O.dampen(H32.astype(np.float64), 0.01)[0])
    Hd = torch.from_numpy(H32).cuda()
    U, info = B.gptq_prepare_hinv(Hd, 0.01, U=Hd)
    torch.cuda.synchronize()
    assert info.tolist() == [0, 0] and U.data_ptr() == Hd.data_ptr()
    assert rel_fro(Hd.cpu().numpy(), Uref) <= TOL_U_FRO
    assert np.array_equal(Hd.cpu().numpy(), np.triu(Hd.cpu().numpy()))


def test_quantize_block_size_invariance_on_gpu(B):
    R, C = 128, 1024
    L = _layer(R, C, 3000, cfg=7)
    W16 = L.w()
    H = O.hessian_accumulate(np.zeros((C, C)), L.x_bits())
    U32 = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0]).astype(np.float32)
    outs = [_run_quant(B, W16, U32, 2, 128, False, blk) for blk in (32, 64, 128, 256)]
    ref = O.quantize_layer(W16, U32.astype(np.float64), 2, 128, False, 128)
    for o in outs:
        check_quantize_outputs(o, ref, W16, 2, C, H)


def test_quantize_degenerate_inputs(B):
    C = 64
    U32 = np.eye(C, dtype=np.float32)
    # all-zero weights: grid [-1, 1], every code = zero-point, loss 0
    out = _run_quant(B, np.zeros((3, C), np.float16), U32, 4, 0, False, 32)
    ref = O.quantize_layer(np.zeros((3, C), np.float16), U32.astype(np.float64), 4, 0, False, 32)
    check_quantize_outputs(out, ref, np.zeros((3, C), np.float16), 4, C)
    assert out["loss"] == 0.0
    # weights already on their own grid are reproduced exactly
    lv = np.random.default_rng(12).integers(0, 16, size=(5, C))
    lv[:, 0], lv[:, 1] = 0, 15
    Wg = ((lv - 8) * 2.0 ** -7).astype(np.float16)
    out = _run_quant(B, Wg, U32, 4, 0, False, 32)
    assert np.array_equal(O.unpack_codes(out["qweight"].view(np.uint32), 4, C), lv) and out["loss"] == 0.0


def test_quantize_reports_nonfinite_weights(B):
    C = 64
    W = np.full((4, C), 0.01, np.float16)
    W[2, 5] = np.inf
    out = B.gptq_quantize_layer(torch.from_numpy(W).cuda(), torch.eye(C, device="cuda"), 4, 0, False, 32)
    torch.cuda.synchronize()
    st, where = out["dev_info"].tolist()
    assert st == B.ERR_NONFINITE and where == 2


def test_argument_errors_are_synchronous(B):
    H = torch.zeros((48, 48), device="cuda")
    X = torch.zeros((4, 48), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.GptqError) as e:
        B.gptq_hessian_accumulate(H, X)          # C % 32 != 0
    assert e.value.status == B.ERR_INVALID_ARG
    W = torch.zeros((4, 64), dtype=torch.float16, device="cuda")
    U = torch.eye(64, device="cuda")
    for kw, st in ((dict(bits=5), B.ERR_UNSUPPORTED), (dict(bits=4, block=48), B.ERR_UNSUPPORTED),
                   (dict(bits=4, group_size=48), B.ERR_INVALID_ARG), (dict(bits=4, block=0), B.ERR_INVALID_ARG),
                   (dict(bits=4, group_size=64, block=96), B.ERR_INVALID_ARG)):      # group and block do not nest
        with pytest.raises(B.GptqError) as e:
            B.gptq_quantize_layer(W, U, **kw)
        assert e.value.status == st


# ------------------------------------------------------------------ end to end, config 0
def test_config0_end_to_end(B, D):
    wl = WL.workload(0)
    L = wl.layers[0]
    grid = wl.grids[0]
    bits_host = L.x_bits()
    W16 = L.w()
    ref = O.solve_layer(W16, bits_host, grid.bits, grid.group_size, grid.sym, wl.block, wl.damp)
    X = D.fill_x(L)
    W = D.fill_w(L)
    H = torch.zeros((L.C, L.C), dtype=torch.float32, device="cuda")
    B.gptq_hessian_accumulate(H, X)
    U, info = B.gptq_prepare_hinv(H, wl.damp)
    out = B.gptq_quantize_layer(W, U, grid.bits, grid.group_size, grid.sym, wl.block)
    torch.cuda.synchronize()
    assert info.tolist()[0] == 0 and out["dev_info"].tolist()[0] == 0
    assert rel_fro(H.cpu().numpy(), ref["H"]) <= TOL_H_FRO
    assert rel_fro(U.cpu().numpy(), ref["U"]) <= TOL_U_FRO
    gpu = dict(qweight=out["qweight"].cpu().numpy(), scales=out["scales"].cpu().numpy(),
               zeros=out["zeros"].cpu().numpy(), loss=out["loss"].item())
    figs = check_quantize_outputs(gpu, ref, W16, grid.bits, L.C, ref["H"])
    print("config0 end-to-end:", figs)


def test_midsize_end_to_end_grouped(B, D):
    """2048 columns, 32768 tokens, 3-bit g128: every stage crosses several outer panels / blocks and all
    tensor-core paths run; the oracle does the whole layer (its own H and U) for the comparison."""
    L = _layer(192, 2048, 32768, cfg=6, kind="fc1")
    bits_host = np.concatenate([L.x_bits(t0, t0 + 8192) for t0 in range(0, L.n_tokens, 8192)])
    W16 = L.w()
    ref = O.solve_layer(W16, bits_host, 3, 128, False, 128, 0.01)
    X, W = D.fill_x(L), D.fill_w(L)
    H = torch.zeros((L.C, L.C), dtype=torch.float32, device="cuda")
    B.gptq_hessian_accumulate(H, X)
    U, info = B.gptq_prepare_hinv(H, 0.01)
    out = B.gptq_quantize_layer(W, U, 3, 128, False, 128)
    torch.cuda.synchronize()
    assert info.tolist()[0] == 0 and out["dev_info"].tolist()[0] == 0
    assert rel_fro(H.cpu().numpy(), ref["H"]) <= TOL_H_FRO
    assert rel_fro(U.cpu().numpy(), ref["U"]) <= TOL_U_FRO
    gpu = dict(qweight=out["qweight"].cpu().numpy(), scales=out["scales"].cpu().numpy(),
               zeros=out["zeros"].cpu().numpy(), loss=out["loss"].item())
    figs = check_quantize_outputs(gpu, ref, W16, 3, L.C, ref["H"])
    print("midsize end-to-end:", figs)


def test_calls_on_a_non_current_stream_with_library_made_temporaries(B):
    """Stages 2 and 3 launched on a stream that is NOT torch's current stream, with the wrapper creating the
    workspace, dev_info and outputs itself, while the current stream keeps allocating and overwriting memory:
    the temporaries must be ordered on the launch stream, so the results still match the oracle."""
    C, R = 1280, 96                                  # two outer panels: stage 2 also uses its internal streams
    L = _layer(R, C, 3000, cfg=5, kind="k")
    W16 = L.w()
    H64 = O.hessian_accumulate(np.zeros((C, C)), L.x_bits())
    H32 = H64.astype(np.float32)
    Uref = O.cholesky_inverse_upper(O.dampen(H32.astype(np.float64), 0.01)[0])
    Hd, Wd = torch.from_numpy(H32).cuda(), torch.from_numpy(W16).cuda()
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    need = max(B.gptq_prepare_hinv_workspace_bytes(C), B.gptq_quantize_workspace_bytes(R, C, 3, 128, 128))
    for _ in range(3):
        U, info = B.gptq_prepare_hinv(Hd, 0.01, stream=side)
        junk = [torch.full((need // 4 + 64,), float("nan"), device="cuda") for _ in range(3)]   # current stream
        out = B.gptq_quantize_layer(Wd, U, 3, 128, False, 128, stream=side)
        junk += [torch.full((need // 4 + 64,), float("nan"), device="cuda") for _ in range(3)]
        junk += [torch.full((16,), -1, dtype=torch.int32, device="cuda") for _ in range(64)]
        side.synchronize()
        torch.cuda.synchronize()
        del junk
        assert info.tolist() == [0, 0] and out["dev_info"].tolist()[0] == 0
        assert rel_fro(U.cpu().numpy(), Uref) <= TOL_U_FRO
        ref = O.quantize_layer(W16, U.cpu().numpy().astype(np.float64), 3, 128, False, 128)
        gpu = dict(qweight=out["qweight"].cpu().numpy(), scales=out["scales"].cpu().numpy(),
                   zeros=out["zeros"].cpu().numpy(), loss=out["loss"].item())
        check_quantize_outputs(gpu, ref, W16, 3, C, H64)


def test_solve_layer_from_host_buffers(B):
    """The host-buffer entry point (X streamed in chunks, results copied back) against the oracle."""
    L = _layer(96, 512, 5000, cfg=5, kind="o")
    bits_host = L.x_bits()
    W16 = L.w()
    ref = O.solve_layer(W16, bits_host, 4, 0, False, 128, 0.01)
    Xh = torch.from_numpy(bits_host.view(np.int16)).view(torch.bfloat16).pin_memory()
    Wh = torch.from_numpy(W16).pin_memory()
    for _ in range(2):                      # twice: the second call reuses the result buffers and workspace
        out = B.gptq_solve_layer_host(Wh, Xh, 4, 0, False, 128, 0.01)
    assert out["info"].tolist() == [0, 0]
    gpu = dict(qweight=out["qweight"].numpy(), scales=out["scales"].numpy(), zeros=out["zeros"].numpy(),
               loss=out["loss"].item())
    check_quantize_outputs(gpu, ref, W16, 4, L.C, ref["H"])
    with pytest.raises(B.GptqError):
        B.gptq_solve_layer_host(Wh, Xh, 5, 0, False, 128, 0.01)      # unsupported bits


def test_two_host_buffer_calls_in_flight_match_the_oracle(B):
    """Two host threads, each with its own stream and device workspace, solve different layers at the same time
    (the benchmark's end-to-end leg does this).  Stage 2 shares its internal streams and events between the calls;
    both results must still match the oracle.  The wider layer has several outer panels, so those streams are used."""
    import threading
    cases = [(_layer(64, 2304, 3000, cfg=7, kind="fc2"), 3, 128), (_layer(96, 1280, 4000, cfg=8, kind="q"), 4, 0)]
    refs, inputs = [], []
    for L, bits, group in cases:
        xb, W16 = L.x_bits(), L.w()
        refs.append((O.solve_layer(W16, xb, bits, group, False, 128, 0.01), W16, bits, L))
        inputs.append((torch.from_numpy(W16).pin_memory(), torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).pin_memory()))
    dev = torch.cuda.current_device()
    outs, errs = [None, None], []

    def work(i):
        try:
            torch.cuda.set_device(dev)
            stream = torch.cuda.Stream()
            _, bits, group = cases[i][0], cases[i][1], cases[i][2]
            for _ in range(3):              # several rounds so that the two calls really overlap
                outs[i] = B.gptq_solve_layer_host(inputs[i][0], inputs[i][1], bits, group, False, 128, 0.01, stream=stream)
        except Exception as e:
            errs.append(e)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errs, errs
    for out, (ref, W16, bits, L) in zip(outs, refs):
        assert out["info"].tolist() == [0, 0]
        gpu = dict(qweight=out["qweight"].numpy(), scales=out["scales"].numpy(), zeros=out["zeros"].numpy(),
                   loss=out["loss"].item())
        check_quantize_outputs(gpu, ref, W16, bits, L.C, ref["H"])


@pytest.mark.parametrize("bits,group", [(4, 0), (3, 0), (3, 128), (2, 32), (4, 8), (4, 1024), (O.BITS_TERNARY, 8), (8, 64)])
def test_rtn_layer_bit_exact_and_equals_solver_on_diagonal_hessian(B, bits, group):
    """RTN entry point: codes, scales and zeros bit-exact against the oracle's RTN (both sides decide in
    fp64 on fp32-rounded scales); and the solver with a diagonal H gives the same codes (Section 5, Baselines)."""
    L = _layer(70, 2048, 64, cfg=4)
    W16 = L.w()
    W = torch.from_numpy(W16).cuda()
    out = B.gptq_rtn_layer(W, bits, group, False)
    torch.cuda.synchronize()
    codes_ref, _ = O.rtn(W16, bits, group, False)
    codes = O.unpack_codes(out["qweight"].cpu().numpy().view(np.uint32), bits, L.C)
    assert np.array_equal(codes, codes_ref)
    assert np.array_equal(O.pack_codes(codes, bits), out["qweight"].cpu().numpy().view(np.uint32))
    g = group if group > 0 else L.C
    for gi in range(0, L.C // g, max(1, (L.C // g) // 7)):
        s, z = O.find_params(W16[:, gi * g:(gi + 1) * g].astype(np.float64), bits, False)
        assert np.array_equal(out["scales"][:, gi].cpu().numpy().astype(np.float64), s)
        assert np.array_equal(out["zeros"][:, gi].cpu().numpy().astype(np.float64), z)
    if group == 0 or (group % 32 == 0) or group in (4, 8, 16):
        d = np.exp(np.random.default_rng(3).normal(size=L.C)).astype(np.float32)
        U, info = B.gptq_prepare_hinv(torch.diag(torch.from_numpy(d)).cuda(), 0.01)
        blk = 128 if (group <= 0 or group % 128 == 0 or 128 % group == 0) else 32
        q = B.gptq_quantize_layer(W, U, bits, group, False, blk)
        torch.cuda.synchronize()
        assert torch.equal(q["qweight"], out["qweight"])


@pytest.mark.parametrize("bits,group,C,sym,fp16", [
    (2, 256, 2304, False, False), (3, 32, 2080, False, False), (3, 64, 2112, False, True), (4, 256, 2304, True, False),
    (8, 256, 1024, False, False), (2, 0, 2080, False, False), (8, 0, 2048, False, False), (3, 96, 2016, False, False),
    (4, 384, 2304, False, True), (2, 160, 2080, True, False), (3, 256, 2304, False, False), (O.BITS_TERNARY, 128, 2176, False, False),
    (4, 16, 2080, False, False), (3, 4, 2080, False, False), (4, 2080, 2080, False, False), (3, 1024, 4096, False, False)])
def test_rtn_layer_every_kind_of_group(B, bits, group, C, sym, fp16):
    """gptq_rtn_layer over the group sizes its three kernels serve: runs of power-of-two groups (32 ... 256, with a last run
    that is not full and a row that is not a multiple of 256 columns), one warp per group (multiples of 32 that are not a
    power of two, groups of several hundred columns, per-row grids) and the small groups (4, 8, 16); symmetric grids and
    fp16-rounded scales included.  Codes, scales and zero-points bit for bit against the oracle."""
    R = 37
    L = _layer(R, C, 64, cfg=14)
    W16 = L.w()
    out = B.gptq_rtn_layer(torch.from_numpy(W16).cuda(), bits, group, sym, scale_fp16=fp16)
    torch.cuda.synchronize()
    codes_ref, _ = O.rtn(W16, bits, group, sym, scale_fp16=fp16)
    codes = O.unpack_codes(out["qweight"].cpu().numpy().view(np.uint32), bits, C)
    assert np.array_equal(codes, codes_ref)
    assert np.array_equal(O.pack_codes(codes, bits), out["qweight"].cpu().numpy().view(np.uint32))
    g = group if group > 0 else C
    grids = [O.find_params(W16[:, j:j + g].astype(np.float64), bits, sym, fp16) for j in range(0, C, g)]
    assert np.array_equal(out["scales"].cpu().numpy().astype(np.float64), np.stack([a for a, _ in grids], 1))
    assert np.array_equal(out["zeros"].cpu().numpy().astype(np.float64), np.stack([b for _, b in grids], 1))


@pytest.mark.parametrize("bits,group,C", [(4, 0, 2048), (3, 128, 2048), (2, 32, 2048), (O.BITS_TERNARY, 8, 2048), (8, 0, 2048),
                                          (3, 0, 2048), (2, 128, 2048), (4, 128, 4096), (4, 1024, 2048), (O.BITS_TERNARY, 0, 2080),
                                          (8, 128, 1024), (3, 0, 2144), (4, 0, 96), (3, 384, 768)])
def test_dequantize_and_matvec_match_oracle(B, bits, group, C):
    """Inference-side kernels on the packed layout: dequantization bit-exact (fp32 product, RNE to fp16);
    matvec within fp32 accumulation error of the fp64 definition.  Per-row grids and groups that are multiples
    of 128 take the tensor-core kernel (ragged last row task, C not a multiple of 128 included), the others the
    CUDA-core kernel."""
    R = 300
    L = _layer(R, C, 64, cfg=3)
    W16 = L.w()
    codes, _ = O.rtn(W16, bits, group, False)
    g = group if group > 0 else C
    scales = np.stack([O.find_params(W16[:, j:j + g].astype(np.float64), bits, False)[0] for j in range(0, C, g)], 1)
    zeros = np.stack([O.find_params(W16[:, j:j + g].astype(np.float64), bits, False)[1] for j in range(0, C, g)], 1)
    qw = torch.from_numpy(O.pack_codes(codes, bits).view(np.int32)).cuda()
    sc = torch.from_numpy(scales.astype(np.float32)).cuda()
    zr = torch.from_numpy(zeros.astype(np.float32)).cuda()
    deq = B.gptq_dequantize(qw, sc, zr, C, bits, group)
    ref16 = O.dequantize(codes, scales, zeros, to_fp16=True)
    assert np.array_equal(deq.cpu().numpy().view(np.uint16), ref16.view(np.uint16))
    x16 = (np.random.default_rng(9).normal(size=C)).astype(np.float16)
    y = B.gptq_matvec(qw, sc, zr, torch.from_numpy(x16).cuda(), C, bits, group).cpu().numpy().astype(np.float64)
    yref = O.matvec(codes, scales, zeros, x16)
    # the kernels form sum q x and zero * sum x separately (fp32, tensor-core accumulators drained every 128 columns),
    # so their rounding error scales with those un-centred sums: 4e-6 of scale * (q + zero) * |x| summed over the row
    gsz = C // scales.shape[1]
    mag = np.repeat(scales, gsz, 1) * (codes + np.repeat(zeros, gsz, 1))
    bound = 4e-6 * (mag @ np.abs(x16.astype(np.float64))) + 1e-12
    assert (np.abs(y - yref) <= bound).all(), float(np.max(np.abs(y - yref) / bound))


@pytest.mark.parametrize("R,C,bits,group", [(5000, 6272, 4, 0), (2500, 12288, 3, 128), (4800, 8256, 2, 0), (2400, 5120, 8, 128),
                                            (37, 4160, 4, 0), (2385, 49152, 4, 0), (2385, 16384, 3, 0), (300, 12288, 2, 128)])
def test_matvec_over_several_row_tasks_and_stages_per_warp(B, bits, group, R, C):
    """The tensor-core matvec with the codes staged through shared memory: more row tasks than CTAs (the rings run
    across task boundaries), several stages per warp and task, a ragged last row task, a last block of 64 or 32 columns,
    and x so long that the rings shrink to fewer stages.  Random codes and grids; oracle: the fp64 definition."""
    r = np.random.default_rng(R + C + bits)
    maxq = O.maxq_of(bits)
    g = group if group > 0 else C
    codes = r.integers(0, maxq + 1, size=(R, C))
    scales = np.exp(r.normal(size=(R, C // g)) * 0.3).astype(np.float32).astype(np.float64) * 0.01
    zeros = r.integers(0, maxq + 1, size=(R, C // g)).astype(np.float64)
    x16 = r.normal(size=C).astype(np.float16)
    qw = torch.from_numpy(O.pack_codes(codes, bits).view(np.int32)).cuda()
    sc, zr = torch.from_numpy(scales.astype(np.float32)).cuda(), torch.from_numpy(zeros.astype(np.float32)).cuda()
    y = B.gptq_matvec(qw, sc, zr, torch.from_numpy(x16).cuda(), C, bits, group).cpu().numpy().astype(np.float64)
    yref = O.matvec(codes, scales.astype(np.float32).astype(np.float64), zeros, x16)
    mag = np.repeat(scales, g, 1) * (codes + np.repeat(zeros, g, 1))
    bound = 4e-6 * (mag @ np.abs(x16.astype(np.float64))) + 1e-12
    assert (np.abs(y - yref) <= bound).all(), float(np.max(np.abs(y - yref) / bound))


def test_matvec_rejects_misaligned_operands(B):
    """x and the packed matrix are read in 16-byte pieces: operands that start elsewhere are refused at the call, before
    anything is launched."""
    R, C, bits = 70, 1024, 4
    packed = torch.zeros(R * C // 8 + 4, dtype=torch.int32, device="cuda")
    sc, zr = torch.ones((R, 1), device="cuda"), torch.zeros((R, 1), device="cuda")
    xbuf = torch.zeros(C + 8, dtype=torch.float16, device="cuda")
    y = torch.empty(R, dtype=torch.float32, device="cuda")
    n0 = B.gptq_launch_count()
    st = B._lib.gptq_matvec(packed.data_ptr(), sc.data_ptr(), zr.data_ptr(), xbuf.data_ptr() + 2, R, C, bits, 0, y.data_ptr(), None)
    assert st == B.ERR_INVALID_ARG
    st = B._lib.gptq_matvec(packed.data_ptr() + 4, sc.data_ptr(), zr.data_ptr(), xbuf.data_ptr(), R, C, bits, 0, y.data_ptr(), None)
    assert st == B.ERR_INVALID_ARG
    assert B.gptq_launch_count() == n0
    assert B._lib.gptq_matvec(packed.data_ptr(), sc.data_ptr(), zr.data_ptr(), xbuf.data_ptr(), R, C, bits, 0, y.data_ptr(), None) == 0
    torch.cuda.synchronize()


def test_block_pipeline_shares_hessian_and_factor_for_q_k_v(B, D):
    """Section 5, Setup: a block's layers are quantized from one pass of calibration inputs.  q, k and v read the same
    input, so the pipeline computes ONE Hessian and ONE factor for them; every member's outputs are bit-identical to
    stages 2-3 run alone on the group's Hessian and agree with a fully separate solve of that layer; o / fc1 / fc2
    keep their own inputs."""
    from paper_2210_17323_b200 import pipeline as P
    C, F, m = 512, 1280, 3000
    layers = [WL.Layer(7, 0, k, C, C, m) for k in ("q", "k", "v", "o")] + [WL.Layer(7, 0, "fc1", F, C, m), WL.Layer(7, 0, "fc2", C, F, m)]
    shared_x = D.fill_x(layers[0])                         # q's input is also k's and v's
    groups = P.group_by_shared_input(layers, lambda L: shared_x if L.kind == "q" else D.fill_x(L), D.fill_w)
    assert [[mm.name for mm in g.members] for g in groups] == [[layers[0].name, layers[1].name, layers[2].name], [layers[3].name],
                                                               [layers[4].name], [layers[5].name]]
    solver = P.BlockSolver(groups, 3, 128, False, 128, 0.01)
    solver.enqueue()
    torch.cuda.synchronize()
    solver.check()
    res = solver.results()
    H_of = {mm["m"].name: st["H"] for st in solver.state for mm in st["members"]}
    assert H_of[layers[0].name] is H_of[layers[1].name] is H_of[layers[2].name]          # one Hessian for q, k, v
    for L in layers:
        # (a) stages 2 and 3 alone from the group's Hessian: bit-identical (they are deterministic at these sizes), so the
        #     pipeline handed the right factor and the right weights to every member
        U, info = B.gptq_prepare_hinv(H_of[L.name], 0.01)
        out = B.gptq_quantize_layer(D.fill_w(L), U, 3, 128, False, 128)
        torch.cuda.synchronize()
        assert info.tolist()[0] == 0
        for key in ("qweight", "scales", "zeros"):
            assert torch.equal(out[key], res[L.name][key]), (L.name, key)
        # (b) a fully separate solve with its own Hessian of the same input: the Hessian kernel adds token ranges with
        #     floating-point reductions whose order varies from run to run, so equality is up to that rounding
        X = shared_x if L.kind in ("q", "k", "v") else D.fill_x(L)
        H = torch.zeros((L.C, L.C), dtype=torch.float32, device="cuda")
        B.gptq_hessian_accumulate(H, X)
        assert rel_fro(H.cpu().numpy(), H_of[L.name].cpu().numpy()) <= 1e-6
        U2, _ = B.gptq_prepare_hinv(H, 0.01)
        out2 = B.gptq_quantize_layer(D.fill_w(L), U2, 3, 128, False, 128)
        torch.cuda.synchronize()
        a = O.unpack_codes(out2["qweight"].cpu().numpy().view(np.uint32), 3, L.C)
        b = O.unpack_codes(res[L.name]["qweight"].cpu().numpy().view(np.uint32), 3, L.C)
        assert (a == b).mean() >= 0.999 and np.abs(a - b).max() <= 1
        assert rel_fro(out2["scales"].cpu().numpy(), res[L.name]["scales"].cpu().numpy()) <= 1e-5
    # and one member against the oracle, end to end
    L = layers[1]
    bits_host = shared_x.view(torch.int16).cpu().numpy().view(np.uint16)
    ref = O.solve_layer(L.w(), bits_host, 3, 128, False, 128, 0.01)
    o = res[L.name]
    gpu = dict(qweight=o["qweight"].cpu().numpy(), scales=o["scales"].cpu().numpy(), zeros=o["zeros"].cpu().numpy(),
               loss=o["loss"].item())
    check_quantize_outputs(gpu, ref, L.w(), 3, L.C, ref["H"])


def test_bounded_waits_report_timeout_and_the_gpu_stays_usable(B, D):
    """Every wait in the tensor-core kernels is bounded.  With the limit lowered to 20 ms and the loads of one work item
    left out (a barrier that nothing completes), the Hessian kernel must come back by itself with GPTQ_ERR_TIMEOUT in
    dev_info -- every role leaving through its own bounded wait, tensor memory freed -- and the next, normal call on the
    same context must work and give the right Hessian."""
    L = _layer(8, 768, 4096, cfg=3)
    X = D.fill_x(L)
    H = torch.zeros((L.C, L.C), dtype=torch.float32, device="cuda")
    info = torch.zeros(2, dtype=torch.int32, device="cuda")
    B.gptq_debug_wait_test(20_000_000, 0)
    try:
        B.gptq_hessian_accumulate(H, X, dev_info=info)
        torch.cuda.synchronize()
        st, where = info.tolist()
        assert st == B.ERR_TIMEOUT and 21 <= where <= 27, (st, where)   # whichever role's wait ran out first
    finally:
        B.gptq_debug_wait_test(0, -1)
    H.zero_()
    B.gptq_hessian_accumulate(H, X, dev_info=info)
    torch.cuda.synchronize()
    assert info.tolist() == [0, 0]
    Href = O.hessian_accumulate(np.zeros((L.C, L.C)), L.x_bits())
    assert rel_fro(H.cpu().numpy(), Href) <= TOL_H_FRO


def test_solve_layer_from_host_buffers_several_grids(B):
    """One host-buffer call for several grids of a layer (activations cross once, one Hessian and factor): every grid's
    result matches the oracle, and equals the single-grid call's for the grid they share."""
    L = _layer(96, 1280, 5000, cfg=5, kind="v")
    bits_host, W16 = L.x_bits(), L.w()
    Xh = torch.from_numpy(bits_host.view(np.int16)).view(torch.bfloat16).pin_memory()
    Wh = torch.from_numpy(W16).pin_memory()
    grids = [(4, 0, False), (3, 128, False), (B.BITS_TERNARY, 32, False)]
    outs = None
    for _ in range(2):                      # twice: the second call reuses the result buffers
        outs = B.gptq_solve_layer_host_grids(Wh, Xh, grids, 128, 0.01, outs=outs)
    assert outs[0]["info"].tolist() == [0, 0]
    H = O.hessian_accumulate(np.zeros((L.C, L.C)), bits_host)
    U = O.cholesky_inverse_upper(O.dampen(H, 0.01)[0])
    for (bits, group, sym), o in zip(grids, outs):
        ref = O.quantize_layer(W16, U, bits, group, sym, 128)
        gpu = dict(qweight=o["qweight"].numpy(), scales=o["scales"].numpy(), zeros=o["zeros"].numpy(), loss=o["loss"].item())
        check_quantize_outputs(gpu, ref, W16, bits, L.C, H)
    single = B.gptq_solve_layer_host(Wh, Xh, 3, 128, False, 128, 0.01)
    a = O.unpack_codes(single["qweight"].numpy().view(np.uint32), 3, L.C)
    b = O.unpack_codes(outs[1]["qweight"].numpy().view(np.uint32), 3, L.C)
    assert (a == b).mean() >= 0.999


def test_solve_layer_host_streams_x_in_growing_chunks(B):
    """gptq_solve_layer_host with more tokens than its first chunks hold (the chunks grow by a quarter each from 1/16 of
    the full chunk; all but the last add to the upper triangle of H only).  Small-integer activations make every sum of the
    Hessian exact, so the result must equal, bit for bit, that of the three device calls on the whole X at once."""
    R, C, n = 48, 2048, 110000                      # full chunk = 2 GiB / (2 C) = 524288 tokens: chunks of 32768, 40960, 36272
    r = np.random.default_rng(21)
    Xi = r.integers(-3, 4, size=(n, C)).astype(np.float32)
    Xi[:, ::7] *= 2.0                               # a spread of channel energies
    Xh = torch.from_numpy(Xi).to(torch.bfloat16).contiguous().pin_memory()
    Wh = torch.from_numpy(_layer(R, C, 64, cfg=15).w()).pin_memory()
    host = B.gptq_solve_layer_host(Wh, Xh, 4, 128, False, 128, 0.01)
    assert host["info"].tolist() == [0, 0]
    H = torch.zeros((C, C), dtype=torch.float32, device="cuda")
    B.gptq_hessian_accumulate(H, Xh.cuda())
    F, info = B.gptq_prepare_hinv(H, 0.01, factor=True)      # the host call takes the factor form for C > 1024
    dev = B.gptq_quantize_layer(Wh.cuda(), F, 4, 128, False, 128, factor=True)
    torch.cuda.synchronize()
    assert info.tolist() == [0, 0] and dev["dev_info"].tolist() == [0, 0]
    assert torch.equal(host["qweight"], dev["qweight"].cpu())
    assert torch.equal(host["scales"], dev["scales"].cpu()) and torch.equal(host["zeros"], dev["zeros"].cpu())


def test_host_layer_solver_matches_the_oracle(B):
    """pipeline.HostLayerSolver: several layers from pinned host buffers in one overlapped schedule (one copy stream,
    Hessians chunk by chunk as the chunks land, every layer's stages 2-3 on its own stream, results back on the host).
    Small chunks so that every Hessian is accumulated over several ragged pieces; every grid of every layer against the
    oracle; a second solve() reuses all buffers."""
    from paper_2210_17323_b200 import pipeline
    cases = [_layer(64, 1280, 3000, cfg=11, kind="fc2"), _layer(96, 512, 2500, cfg=12, kind="q"), _layer(40, 768, 1000, cfg=13, kind="o")]
    grids = [(4, 0, False), (3, 128, False)]
    layers, refs = [], []
    for L in cases:
        xb, W16 = L.x_bits(), L.w()
        layers.append((torch.from_numpy(W16).pin_memory(), torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).pin_memory()))
        refs.append([O.solve_layer(W16, xb, b, g, s, 128, 0.01) for (b, g, s) in grids])
    solver = pipeline.HostLayerSolver([(L.R, L.C, L.n_tokens) for L in cases], grids, block=128, damp=0.01, chunk_bytes=1 << 20)
    assert any(len(st["chunks"]) > 2 for st in solver.state)
    for _ in range(2):
        outs = solver.solve(layers)
    for L, (Wh, _), per_grid, ref_grids in zip(cases, layers, outs, refs):
        for (b, g, s), out, ref in zip(grids, per_grid, ref_grids):
            assert out["info"].tolist() == [0, 0]
            gpu = dict(qweight=out["qweight"].numpy(), scales=out["scales"].numpy(), zeros=out["zeros"].numpy(),
                       loss=out["loss"].item())
            check_quantize_outputs(gpu, ref, Wh.numpy(), b, L.C, ref["H"])


def test_two_hessian_launches_side_by_side_on_two_streams(B):
    """Two Hessian accumulations of different shapes enqueued on two streams at once.  Each launch hands its work items
    out among its own running clusters (a cluster takes over the items of clusters of ITS grid that have not started);
    with both grids resident at the same time every item must still be done exactly once: on integer-valued inputs the
    results are exact, so one lost or repeated item would show."""
    r = np.random.default_rng(11)
    shapes = [(1280, 9000), (768, 20000)]
    Xs = [torch.from_numpy(r.integers(-4, 5, size=(m, C)).astype(np.float32)).cuda().to(torch.bfloat16) for C, m in shapes]
    Hs = [torch.zeros((C, C), dtype=torch.float32, device="cuda") for C, _ in shapes]
    infos = [torch.zeros(2, dtype=torch.int32, device="cuda") for _ in shapes]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for rep in range(3):                      # three rounds: 3 x the exact sum
        for X, H, info, s in zip(Xs, Hs, infos, streams):
            with torch.cuda.stream(s):
                B.gptq_hessian_accumulate(H, X, dev_info=info)
    torch.cuda.synchronize()
    for X, H, info in zip(Xs, Hs, infos):
        assert info.tolist() == [0, 0]
        Xd = X.double()
        exact = (6.0 * (Xd.T @ Xd)).cpu().numpy()
        assert np.array_equal(H.cpu().numpy().astype(np.float64), exact)


# ------------------------------------------------------------------ factor form (stage 2 without the inverse)
def test_prepare_factor_holds_the_factor_above_and_u_on_the_diagonal_blocks(B):
    """gptq_prepare_factor against the oracle: diagonal blocks of 1024 columns = the blocks of U; above a diagonal block
    J the factor's block column times that diagonal block, U~[:j0, J] U_JJ with U~ = U^-1 the upper factor of the damped
    Hessian."""
    C = 2304
    L = _layer(8, C, 2 * C + 100)
    H64 = O.hessian_accumulate(np.zeros((C, C)), L.x_bits())
    F, info = B.gptq_prepare_hinv(torch.from_numpy(H64.astype(np.float32)).cuda(), 0.01, factor=True)
    torch.cuda.synchronize()
    assert info.tolist() == [0, 0]
    Fg = F.cpu().numpy().astype(np.float64)
    U = O.cholesky_inverse_upper(O.dampen(H64.astype(np.float32).astype(np.float64), 0.01)[0])
    Ut = np.linalg.inv(U)
    assert np.array_equal(Fg, np.triu(Fg))
    for j0 in range(0, C, 1024):
        j1 = min(C, j0 + 1024)
        assert rel_fro(Fg[j0:j1, j0:j1], U[j0:j1, j0:j1]) <= TOL_U_FRO
        if j0 > 0:
            assert rel_fro(Fg[:j0, j0:j1], Ut[:j0, j0:j1] @ U[j0:j1, j0:j1]) <= TOL_U_FRO


@pytest.mark.parametrize("R,C,bits,group,block", [(200, 2304, 4, 0, 128), (130, 3072, 3, 128, 128), (96, 2048, 2, 32, 64),
                                                  (64, 2304, O.BITS_TERNARY, 8, 32), (100, 2048, 4, 1024, 256), (70, 768, 4, 0, 128),
                                                  (1, 1056, 4, 0, 128), (129, 1280, 3, 64, 32), (33, 4128, 8, 0, 128)])
def test_factor_form_matches_the_oracle(B, R, C, bits, group, block):
    """Stages 2 and 3 in the factor form (no inverse; plain residuals fed back through the factor across blocks of 1024
    columns) against the oracle, which runs Algorithm 1 as written with U."""
    L = _layer(R, C, 2 * C + 64, cfg=9)
    xb, W16 = L.x_bits(), L.w()
    ref = O.solve_layer(W16, xb, bits, group, False, block, 0.01)
    H = torch.from_numpy(ref["H"].astype(np.float32)).cuda()
    F, info = B.gptq_prepare_hinv(H, 0.01, factor=True)
    out = B.gptq_quantize_layer(torch.from_numpy(W16).cuda(), F, bits, group, False, block, factor=True)
    torch.cuda.synchronize()
    assert info.tolist() == [0, 0] and out["dev_info"].tolist() == [0, 0]
    gpu = dict(qweight=out["qweight"].cpu().numpy(), scales=out["scales"].cpu().numpy(), zeros=out["zeros"].cpu().numpy(),
               loss=out["loss"].item())
    check_quantize_outputs(gpu, ref, W16, bits, C, ref["H"])


def test_factor_form_rejects_blockings_it_cannot_run(B):
    W = torch.zeros((32, 2304), dtype=torch.float16, device="cuda")
    F = torch.eye(2304, device="cuda")
    with pytest.raises(B.GptqError) as e:
        B.gptq_quantize_layer(W, F, 4, 0, False, 96, factor=True)      # outer blocks of 960 columns
    assert e.value.status == B.ERR_UNSUPPORTED


def test_factor_form_with_symmetric_grid_and_fp16_scales(B):
    """The grid options reach the factor form unchanged: symmetric grid and fp16-rounded scales, three outer blocks.
    (With fp32 scales the symmetric grid has a built-in tie: the weight of largest magnitude in a group, when negative,
    sits exactly between codes 0 and 1, and the rounding of the scale decides; fp16 rounding moves it off the tie.)"""
    L = _layer(90, 2304, 5000, cfg=10)
    xb, W16 = L.x_bits(), L.w()
    H64 = O.hessian_accumulate(np.zeros((L.C, L.C)), xb)
    Ht, _ = O.dampen(H64.astype(np.float32).astype(np.float64), 0.01)
    U = O.cholesky_inverse_upper(Ht)
    ref = O.quantize_layer(W16, U, 3, 128, True, 128, scale_fp16=True)
    F, info = B.gptq_prepare_hinv(torch.from_numpy(H64.astype(np.float32)).cuda(), 0.01, factor=True)
    out = B.gptq_quantize_layer(torch.from_numpy(W16).cuda(), F, 3, 128, True, 128, scale_fp16=True, factor=True)
    torch.cuda.synchronize()
    assert info.tolist() == [0, 0] and out["dev_info"].tolist() == [0, 0]
    gpu = dict(qweight=out["qweight"].cpu().numpy(), scales=out["scales"].cpu().numpy(), zeros=out["zeros"].cpu().numpy(),
               loss=out["loss"].item())
    check_quantize_outputs(gpu, ref, W16, 3, L.C, H64, scale_fp16=True)


@pytest.mark.parametrize("factor", [False, True])
def test_symmetric_grid_with_fp32_scales_differs_only_after_its_tie(B, factor):
    """The symmetric grid has a tie by construction: scale = 2a / maxq with a = max |w| of the group and an even number of
    levels put -a exactly midway between codes 0 and 1.  When the weight of largest magnitude is negative and sits in the
    group's first column (it is quantized before any feedback moves it), the fp32 rounding of the scale decides, and that
    rounding follows the last bits of a working weight the two sides hold to ~1e-7.  Both codes are equally near, so the
    check is: rows that never meet the tie are identical; every other row first differs at a group's first column, by the
    0/1 pair; and the loss agrees."""
    g, bits = 128, 3
    L = _layer(90, 2304, 5000, cfg=10)
    W16 = L.w()
    H64 = O.hessian_accumulate(np.zeros((L.C, L.C)), L.x_bits())
    Ht, _ = O.dampen(H64.astype(np.float32).astype(np.float64), 0.01)
    ref = O.quantize_layer(W16, O.cholesky_inverse_upper(Ht), bits, g, True, 128)
    F, info = B.gptq_prepare_hinv(torch.from_numpy(H64.astype(np.float32)).cuda(), 0.01, factor=factor)
    out = B.gptq_quantize_layer(torch.from_numpy(W16).cuda(), F, bits, g, True, 128, factor=factor)
    torch.cuda.synchronize()
    assert info.tolist() == [0, 0] and out["dev_info"].tolist() == [0, 0]
    codes = O.unpack_codes(out["qweight"].cpu().numpy().view(np.uint32), bits, L.C)
    same = codes == ref["codes"]
    scales = out["scales"].cpu().numpy()
    assert same.mean() >= 0.99 and same.all(axis=1).mean() >= 0.85
    for r in range(L.R):
        j = L.C if same[r].all() else int(np.argmin(same[r]))
        if j < L.C:
            assert j % g == 0 and j >= g, f"row {r} first differs at column {j}, not at a group's first column"
            assert {int(codes[r, j]), int(ref["codes"][r, j])} == {0, 1}
        n = min(j // g + 1, L.C // g)            # the groups whose grids were drawn before the row met the tie
        assert rel_fro(scales[r, :n], ref["scales"][r, :n]) <= 1e-5
    assert abs(out["loss"].item() - ref["loss"]) <= 0.01 * ref["loss"]

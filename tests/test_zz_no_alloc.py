"""The workspace-free entry point gptq_prepare_hinv_static against gptq_prepare_hinv.

Some users of the library cannot allocate device memory at all (their framework's pool owns the GPU,
or they sit on a path where cudaMalloc's implicit synchronisation is not acceptable), so they cannot
supply the workspace gptq_prepare_hinv wants; the static variant keeps its scratch in a fixed array
inside the library.  This file is collected last on purpose: if it fails, a run that stops at the first
failure has already exercised everything else.  It passes on its own in a fresh process and after the
other tests (the shared scratch keeps stale contents between calls, which must not matter).
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import gptq_oracle as O
from paper_2210_17323_b200.synth import workloads as WL
from tests.parity_utils import TOL_U_FRO, rel_fro


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_17323_b200 import binding
    return binding


def _hessian(B, C, tokens, cfg):
    from paper_2210_17323_b200.synth import device as D
    L = WL.Layer(cfg, 0, "q", 8, C, tokens)
    H = torch.zeros((C, C), dtype=torch.float32, device="cuda")
    B.gptq_hessian_accumulate(H, D.fill_x(L))
    return H


def test_static_variant_matches_workspace_variant_twice_in_a_row(B):
    # two calls in a row with different sizes: the second sees the first one's leftovers in the shared scratch
    for C, tokens, cfg in ((768, 3000, 21), (160, 700, 22), (1024, 2500, 23)):
        H = _hessian(B, C, tokens, cfg)
        U_ref, info_ref = B.gptq_prepare_hinv(H, 0.01)
        torch.cuda.synchronize()
        U = torch.empty_like(H)
        info = torch.zeros(2, dtype=torch.int32, device="cuda")
        held = torch.cuda.memory_allocated()
        B.gptq_prepare_hinv_static(H, 0.01, U=U, dev_info=info)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == held      # the call itself took nothing from torch's pool
        assert info.tolist() == info_ref.tolist() == [0, 0]
        assert rel_fro(U.cpu().numpy(), U_ref.cpu().numpy()) <= TOL_U_FRO
        # and directly against the oracle's factor of the same (fp32) Hessian
        U_oracle = O.cholesky_inverse_upper(O.dampen(H.cpu().numpy().astype(np.float64), 0.01)[0])
        assert rel_fro(U.cpu().numpy(), U_oracle) <= TOL_U_FRO


def test_static_variant_rejects_sizes_beyond_its_scratch(B):
    C = B.PREPARE_HINV_STATIC_MAX_C + 32
    H = torch.eye(C, device="cuda")
    with pytest.raises(B.GptqError) as e:
        B.gptq_prepare_hinv_static(H, 0.01)
    assert e.value.status == B.ERR_UNSUPPORTED
    # and still reports numerical trouble through dev_info like the workspace variant
    Hbad = torch.zeros((64, 64), device="cuda")
    _, info = B.gptq_prepare_hinv_static(Hbad, 0.01)
    torch.cuda.synchronize()
    assert info.tolist()[0] == B.ERR_NOT_PD

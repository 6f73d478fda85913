"""Thin ctypes binding over libgptq_b200.so: argument marshalling only.

Every step of the solver runs in the CUDA library; torch is used for device memory and
streams.  Loading fails loudly if the library has not been built -- there is no fallback.
Function names and argument order follow include/gptq_b200.h.
"""
from __future__ import annotations

import contextlib
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libgptq_b200.so")

BITS_TERNARY = -1
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NOT_PD, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE = range(8)

from .binding_symbols import EXPORTS  # noqa: E402,F401


class GptqError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__(f"{where}: {status_string(status)} ({int(status)})")


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2210_17323_b200.build` "
            "(the solver has no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    c = ctypes
    lib.gptq_status_string.restype = c.c_char_p
    lib.gptq_status_string.argtypes = [c.c_int]
    lib.gptq_launch_count.restype = c.c_uint64
    lib.gptq_launch_count.argtypes = []
    lib.gptq_debug_wait_test.restype = c.c_int
    lib.gptq_debug_wait_test.argtypes = [c.c_uint64, c.c_int]
    lib.gptq_hessian_workspace_bytes.restype = c.c_size_t
    lib.gptq_hessian_workspace_bytes.argtypes = [c.c_int, c.c_int64]
    lib.gptq_hessian_accumulate.restype = c.c_int
    lib.gptq_hessian_accumulate.argtypes = [c.c_void_p, c.c_void_p, c.c_int64, c.c_int, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p]
    lib.gptq_hessian_accumulate_upper.restype = c.c_int
    lib.gptq_hessian_accumulate_upper.argtypes = lib.gptq_hessian_accumulate.argtypes
    lib.gptq_hessian_symmetrize.restype = c.c_int
    lib.gptq_hessian_symmetrize.argtypes = [c.c_void_p, c.c_int, c.c_void_p]
    lib.gptq_prepare_hinv_workspace_bytes.restype = c.c_size_t
    lib.gptq_prepare_hinv_workspace_bytes.argtypes = [c.c_int]
    lib.gptq_prepare_hinv.restype = c.c_int
    lib.gptq_prepare_hinv.argtypes = [c.c_void_p, c.c_float, c.c_int, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p]
    lib.gptq_prepare_factor.restype = c.c_int
    lib.gptq_prepare_factor.argtypes = lib.gptq_prepare_hinv.argtypes
    lib.gptq_prepare_hinv_static.restype = c.c_int
    lib.gptq_prepare_hinv_static.argtypes = [c.c_void_p, c.c_float, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p]
    lib.gptq_quantize_workspace_bytes.restype = c.c_size_t
    lib.gptq_quantize_workspace_bytes.argtypes = [c.c_int] * 5
    lib.gptq_quantize_layer.restype = c.c_int
    lib.gptq_quantize_layer.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_int, c.c_int, c.c_int,
                                        c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
                                        c.c_void_p, c.c_size_t, c.c_void_p, c.c_void_p]
    lib.gptq_quantize_layer_factor.restype = c.c_int
    lib.gptq_quantize_layer_factor.argtypes = lib.gptq_quantize_layer.argtypes
    lib.gptq_set_stage3_variant.restype = c.c_int
    lib.gptq_set_stage3_variant.argtypes = [c.c_int]
    lib.gptq_solve_layer_host_workspace_bytes.restype = c.c_size_t
    lib.gptq_solve_layer_host_workspace_bytes.argtypes = [c.c_int, c.c_int, c.c_int64, c.c_int, c.c_int, c.c_int]
    lib.gptq_solve_layer_host.restype = c.c_int
    lib.gptq_solve_layer_host.argtypes = [c.c_void_p, c.c_void_p, c.c_int64, c.c_int, c.c_int, c.c_float, c.c_int, c.c_int,
                                          c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
                                          c.c_void_p, c.c_size_t, c.c_void_p]
    lib.gptq_solve_layer_host_grids_workspace_bytes.restype = c.c_size_t
    lib.gptq_solve_layer_host_grids_workspace_bytes.argtypes = [c.c_int, c.c_int, c.c_int64, c.c_int, c.c_void_p, c.c_void_p, c.c_int]
    lib.gptq_solve_layer_host_grids.restype = c.c_int
    lib.gptq_solve_layer_host_grids.argtypes = [c.c_void_p, c.c_void_p, c.c_int64, c.c_int, c.c_int, c.c_float, c.c_int, c.c_void_p,
                                                c.c_void_p, c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
                                                c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p]
    lib.gptq_rtn_layer.restype = c.c_int
    lib.gptq_rtn_layer.argtypes = [c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
    lib.gptq_dequantize.restype = c.c_int
    lib.gptq_dequantize.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p]
    lib.gptq_matvec.restype = c.c_int
    lib.gptq_matvec.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p]
    return lib


_lib = _load()


def status_string(status) -> str:
    return _lib.gptq_status_string(int(status)).decode()


def gptq_launch_count() -> int:
    return int(_lib.gptq_launch_count())


def gptq_debug_wait_test(wait_limit_ns=0, skip_loads_of_item=-1):
    """Test hook: limit of the kernels' bounded waits and one work item whose loads are left out; (0, -1) restores."""
    st = _lib.gptq_debug_wait_test(int(wait_limit_ns), int(skip_loads_of_item))
    if st != OK:
        raise GptqError(st, "gptq_debug_wait_test")


def _stream_ptr(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


@contextlib.contextmanager
def _alloc_on(stream):
    """Temporaries and outputs a wrapper creates (workspace, dev_info, result tensors) are allocated
    and initialised with `stream` current, so torch's caching allocator orders their reuse, and their
    zero-fill, on the stream the library's kernels run on -- not on whatever stream is current."""
    if stream is None:
        yield
    else:
        with torch.cuda.stream(stream):
            yield


def _check(t, dtype, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")


def _ws(nbytes, device, ws):
    if ws is not None and ws.numel() * ws.element_size() >= nbytes:
        return ws
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def field_bits(bits: int) -> int:
    return 2 if bits == BITS_TERNARY else bits


def gptq_hessian_workspace_bytes(C, n_tokens):
    return _lib.gptq_hessian_workspace_bytes(C, n_tokens)


def gptq_prepare_hinv_workspace_bytes(C):
    return _lib.gptq_prepare_hinv_workspace_bytes(C)


def gptq_quantize_workspace_bytes(R, C, bits, group_size, block):
    return _lib.gptq_quantize_workspace_bytes(R, C, bits, group_size, block)


def gptq_hessian_accumulate(H, X, n_tokens=None, ws=None, dev_info=None, stream=None, upper_only=False):
    """H += 2 X^T X for token-major bf16 X (n_tokens x C).  H: C x C fp32, zeroed by the caller first.
    upper_only: gptq_hessian_accumulate_upper (a chunk that is not the last one: the lower triangle stays stale)."""
    with _alloc_on(stream):
        _check(H, torch.float32, "H")
        _check(X, torch.bfloat16, "X")
        C = H.shape[0]
        n = X.shape[0] if n_tokens is None else int(n_tokens)
        ws = _ws(_lib.gptq_hessian_workspace_bytes(C, n), H.device, ws)
        fn = _lib.gptq_hessian_accumulate_upper if upper_only else _lib.gptq_hessian_accumulate
        st = fn(H.data_ptr(), X.data_ptr(), n, C, ws.data_ptr(), ws.numel(),
                None if dev_info is None else dev_info.data_ptr(), _stream_ptr(stream))
        if st != OK:
            raise GptqError(st, "gptq_hessian_accumulate")
        return H


def gptq_hessian_symmetrize(H, stream=None):
    """Copies the upper triangle of H onto the lower one (after chunks added with upper_only=True)."""
    _check(H, torch.float32, "H")
    st = _lib.gptq_hessian_symmetrize(H.data_ptr(), H.shape[0], _stream_ptr(stream))
    if st != OK:
        raise GptqError(st, "gptq_hessian_symmetrize")
    return H


def gptq_prepare_hinv(H, damp=0.01, U=None, ws=None, dev_info=None, stream=None, factor=False):
    """U = Cholesky((H + damp*mean(diag H) I)^-1)^T.  Returns (U, dev_info); dev_info is read by the caller after a sync.
    factor=True calls gptq_prepare_factor instead: the result holds U on its diagonal blocks of 1024 columns and the
    upper factor of the damped H above them, the input of gptq_quantize_layer(..., factor=True)."""
    with _alloc_on(stream):
        _check(H, torch.float32, "H")
        C = H.shape[0]
        U = torch.empty_like(H) if U is None else U
        _check(U, torch.float32, "U")
        dev_info = torch.zeros(2, dtype=torch.int32, device=H.device) if dev_info is None else dev_info
        ws = _ws(_lib.gptq_prepare_hinv_workspace_bytes(C), H.device, ws)
        st = (_lib.gptq_prepare_factor if factor else _lib.gptq_prepare_hinv)(H.data_ptr(), float(damp), C, U.data_ptr(), ws.data_ptr(), ws.numel(),
                                    dev_info.data_ptr(), _stream_ptr(stream))
        if st != OK:
            raise GptqError(st, "gptq_prepare_hinv")
        return U, dev_info


PREPARE_HINV_STATIC_MAX_C = 1024


def gptq_prepare_hinv_static(H, damp=0.01, U=None, dev_info=None, stream=None):
    """gptq_prepare_hinv without a workspace, for callers that cannot allocate device memory
    (memory owned by a framework pool, allocation-free latency paths, fixed budgets): the scratch is
    a fixed 1 MiB array inside the library.  C <= 1024.  All calls on a device share that array, so
    calls that could overlap on the GPU must be put on one stream.  The first call on a device does a
    one-time address look-up and should not happen inside a stream capture.  U and dev_info are the
    caller's (created here with torch only when not passed in)."""
    with _alloc_on(stream):
        _check(H, torch.float32, "H")
        C = H.shape[0]
        U = torch.empty_like(H) if U is None else U
        _check(U, torch.float32, "U")
        dev_info = torch.zeros(2, dtype=torch.int32, device=H.device) if dev_info is None else dev_info
        st = _lib.gptq_prepare_hinv_static(H.data_ptr(), float(damp), C, U.data_ptr(), dev_info.data_ptr(), _stream_ptr(stream))
        if st != OK:
            raise GptqError(st, "gptq_prepare_hinv_static")
        return U, dev_info


GRID_SYMMETRIC, GRID_FP16_SCALES = 1, 2


def _grid_flags(sym, scale_fp16):
    return (GRID_SYMMETRIC if sym else 0) | (GRID_FP16_SCALES if scale_fp16 else 0)


def gptq_quantize_layer(W, U, bits, group_size=0, sym=False, block=128, ws=None, dev_info=None, stream=None, scale_fp16=False,
                        factor=False):
    """Algorithm 1 on fp16 W (R x C) with U from gptq_prepare_hinv (factor=True: gptq_quantize_layer_factor on the
    output of gptq_prepare_hinv(..., factor=True)).
    Returns dict(qweight uint32 [R, C*f/32] (as int32 tensor), scales [R,G], zeros [R,G], loss double[1], dev_info)."""
    with _alloc_on(stream):
        _check(W, torch.float16, "W")
        _check(U, torch.float32, "U")
        R, C = W.shape
        G = C // group_size if group_size > 0 else 1
        f = field_bits(bits)
        dev = W.device
        qweight = torch.empty((R, C * f // 32), dtype=torch.int32, device=dev)
        scales = torch.empty((R, G), dtype=torch.float32, device=dev)
        zeros = torch.empty((R, G), dtype=torch.float32, device=dev)
        loss = torch.zeros(1, dtype=torch.float64, device=dev)
        dev_info = torch.zeros(2, dtype=torch.int32, device=dev) if dev_info is None else dev_info
        ws = _ws(_lib.gptq_quantize_workspace_bytes(R, C, bits, group_size, block), dev, ws)
        st = (_lib.gptq_quantize_layer_factor if factor else _lib.gptq_quantize_layer)(W.data_ptr(), U.data_ptr(), R, C, bits, group_size, _grid_flags(sym, scale_fp16), block,
                                      qweight.data_ptr(), scales.data_ptr(), zeros.data_ptr(), loss.data_ptr(),
                                      ws.data_ptr(), ws.numel(), dev_info.data_ptr(), _stream_ptr(stream))
        if st != OK:
            raise GptqError(st, "gptq_quantize_layer")
        return dict(qweight=qweight, scales=scales, zeros=zeros, loss=loss, dev_info=dev_info)


def factor_form_supported(C, block, group_sizes=()):
    """True if gptq_quantize_layer(..., factor=True) can run this layer: outer blocks of 1024 columns."""
    if C <= 1024:
        return True
    return all(1024 % max(block, g if g and g > 0 else 0) == 0 for g in (list(group_sizes) or [0]))


def factor_form_pays(R, C, n_grids=1):
    """The factor form leaves out the rows of the inverse (about C^3 / 3 multiply-adds) and adds one 1024-deep product per
    block column of the factor (C^2 * 512): it pays for every layer with more than one block of 1024 columns."""
    return C > 1024


def gptq_set_stage3_variant(variant: int) -> int:
    """1: row-stripe kernel inside an outer block (default); 0: per-inner-block kernels.  Returns the previous value."""
    return int(_lib.gptq_set_stage3_variant(int(variant)))


def gptq_solve_layer_host_workspace_bytes(R, C, n_tokens, bits, group_size, block):
    return _lib.gptq_solve_layer_host_workspace_bytes(R, C, n_tokens, bits, group_size, block)


def gptq_solve_layer_host(W_host, X_host, bits, group_size=0, sym=False, block=128, damp=0.01, out=None, dev_ws=None,
                          stream=None):
    """Stages 1-3 for one layer with HOST inputs and outputs (CPU tensors; pinned for overlapped copies).
    Returns dict(qweight int32 [R, C*f/32], scales, zeros, loss float64[1], info int32[2]) of CPU tensors
    (pass `out` to reuse pinned result buffers).  Synchronises the stream."""
    for t, dt, name in ((W_host, torch.float16, "W_host"), (X_host, torch.bfloat16, "X_host")):
        if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.is_contiguous() and t.dtype == dt):
            raise TypeError(f"{name}: expected a contiguous CPU tensor of {dt}")
    R, C = W_host.shape
    n = X_host.shape[0]
    G = C // group_size if group_size > 0 else 1
    f = field_bits(bits)
    if out is None:
        out = dict(qweight=torch.empty((R, C * f // 32), dtype=torch.int32).pin_memory(),
                   scales=torch.empty((R, G), dtype=torch.float32).pin_memory(),
                   zeros=torch.empty((R, G), dtype=torch.float32).pin_memory(),
                   loss=torch.zeros(1, dtype=torch.float64).pin_memory(),
                   info=torch.zeros(2, dtype=torch.int32).pin_memory())
    need = _lib.gptq_solve_layer_host_workspace_bytes(R, C, n, bits, group_size, block)
    if need == 0:
        raise GptqError(ERR_UNSUPPORTED, "gptq_solve_layer_host_workspace_bytes")
    dev_ws = _ws(need, torch.device("cuda", torch.cuda.current_device()), dev_ws)
    st = _lib.gptq_solve_layer_host(W_host.data_ptr(), X_host.data_ptr(), n, R, C, float(damp), bits, group_size,
                                    int(bool(sym)), block, out["qweight"].data_ptr(), out["scales"].data_ptr(),
                                    out["zeros"].data_ptr(), out["loss"].data_ptr(), out["info"].data_ptr(),
                                    dev_ws.data_ptr(), dev_ws.numel(), _stream_ptr(stream))
    if st != OK:
        raise GptqError(st, "gptq_solve_layer_host")
    return out


def gptq_solve_layer_host_grids(W_host, X_host, grids, block=128, damp=0.01, outs=None, dev_ws=None, stream=None):
    """Stages 1-3 for one layer and SEVERAL grids with HOST inputs and outputs: X crosses to the device once, one Hessian
    and one factor serve every grid.  grids: sequence of (bits, group_size, sym) or (bits, group_size, sym, scale_fp16).
    Returns a list of dicts like gptq_solve_layer_host's (pass `outs` to reuse pinned result buffers); the list's first
    dict also carries 'info' (int32[2]).  Synchronises the stream."""
    for t, dt, name in ((W_host, torch.float16, "W_host"), (X_host, torch.bfloat16, "X_host")):
        if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.is_contiguous() and t.dtype == dt):
            raise TypeError(f"{name}: expected a contiguous CPU tensor of {dt}")
    R, C = W_host.shape
    n = X_host.shape[0]
    ng = len(grids)
    c = ctypes
    bits = (c.c_int * ng)(*[g[0] for g in grids])
    group = (c.c_int * ng)(*[g[1] for g in grids])
    sym = (c.c_int * ng)(*[_grid_flags(g[2], g[3] if len(g) > 3 else False) for g in grids])
    if outs is None:
        outs = []
        for g in grids:
            G = C // g[1] if g[1] > 0 else 1
            outs.append(dict(qweight=torch.empty((R, C * field_bits(g[0]) // 32), dtype=torch.int32).pin_memory(),
                             scales=torch.empty((R, G), dtype=torch.float32).pin_memory(),
                             zeros=torch.empty((R, G), dtype=torch.float32).pin_memory()))
        outs[0]["loss_all"] = torch.zeros(ng, dtype=torch.float64).pin_memory()
        outs[0]["info"] = torch.zeros(2, dtype=torch.int32).pin_memory()
    qp = (c.c_void_p * ng)(*[o["qweight"].data_ptr() for o in outs])
    sp = (c.c_void_p * ng)(*[o["scales"].data_ptr() for o in outs])
    zp = (c.c_void_p * ng)(*[o["zeros"].data_ptr() for o in outs])
    need = _lib.gptq_solve_layer_host_grids_workspace_bytes(R, C, n, ng, bits, group, block)
    if need == 0:
        raise GptqError(ERR_UNSUPPORTED, "gptq_solve_layer_host_grids_workspace_bytes")
    dev_ws = _ws(need, torch.device("cuda", torch.cuda.current_device()), dev_ws)
    st = _lib.gptq_solve_layer_host_grids(W_host.data_ptr(), X_host.data_ptr(), n, R, C, float(damp), ng, bits, group, sym, block,
                                          qp, sp, zp, outs[0]["loss_all"].data_ptr(), outs[0]["info"].data_ptr(),
                                          dev_ws.data_ptr(), dev_ws.numel(), _stream_ptr(stream))
    if st != OK:
        raise GptqError(st, "gptq_solve_layer_host_grids")
    for i, o in enumerate(outs):
        o["loss"] = outs[0]["loss_all"][i:i + 1]
    return outs


def gptq_rtn_layer(W, bits, group_size=0, sym=False, stream=None, scale_fp16=False):
    """Round-to-nearest on the solver's grid, no error feedback.  Returns dict(qweight, scales, zeros)."""
    with _alloc_on(stream):
        _check(W, torch.float16, "W")
        R, C = W.shape
        G = C // group_size if group_size > 0 else 1
        qweight = torch.empty((R, C * field_bits(bits) // 32), dtype=torch.int32, device=W.device)
        scales = torch.empty((R, G), dtype=torch.float32, device=W.device)
        zeros = torch.empty((R, G), dtype=torch.float32, device=W.device)
        st = _lib.gptq_rtn_layer(W.data_ptr(), R, C, bits, group_size, _grid_flags(sym, scale_fp16), qweight.data_ptr(), scales.data_ptr(),
                                 zeros.data_ptr(), _stream_ptr(stream))
        if st != OK:
            raise GptqError(st, "gptq_rtn_layer")
        return dict(qweight=qweight, scales=scales, zeros=zeros)


def gptq_dequantize(qweight, scales, zeros, C, bits, group_size=0, out=None, stream=None):
    """Packed codes -> fp16 weights W^ = scales * (code - zeros)  [R x C]."""
    with _alloc_on(stream):
        _check(qweight, torch.int32, "qweight"); _check(scales, torch.float32, "scales"); _check(zeros, torch.float32, "zeros")
        R = qweight.shape[0]
        out = torch.empty((R, C), dtype=torch.float16, device=qweight.device) if out is None else out
        st = _lib.gptq_dequantize(qweight.data_ptr(), scales.data_ptr(), zeros.data_ptr(), R, C, bits, group_size,
                                  out.data_ptr(), _stream_ptr(stream))
        if st != OK:
            raise GptqError(st, "gptq_dequantize")
        return out


def gptq_matvec(qweight, scales, zeros, x, C, bits, group_size=0, out=None, stream=None):
    """y = W^ x for one fp16 vector x of length C, dequantizing on the fly; y is fp32 [R]."""
    with _alloc_on(stream):
        _check(qweight, torch.int32, "qweight"); _check(scales, torch.float32, "scales"); _check(zeros, torch.float32, "zeros")
        _check(x, torch.float16, "x")
        R = qweight.shape[0]
        out = torch.empty(R, dtype=torch.float32, device=qweight.device) if out is None else out
        st = _lib.gptq_matvec(qweight.data_ptr(), scales.data_ptr(), zeros.data_ptr(), x.data_ptr(), R, C, bits, group_size,
                              out.data_ptr(), _stream_ptr(stream))
        if st != OK:
            raise GptqError(st, "gptq_matvec")
        return out

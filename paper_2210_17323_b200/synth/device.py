"""Device-side filler for the seeded synthetic inputs (torch tensors on the GPU).

Bit-identical to generator.py (checked by the GPU tests); used where the host
generator would take too long (hundreds of millions of activations and more).
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

from . import generator as G

_LIB_PATH = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "lib", "libgptq_synth.so")
_lib = None
_tables = {}


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2210_17323_b200.build`")
        _lib = ctypes.CDLL(_LIB_PATH)
        c = ctypes
        _lib.synth_fill_x_bf16.restype = c.c_int
        _lib.synth_fill_x_bf16.argtypes = [c.c_void_p, c.c_int64, c.c_int, c.c_int64, c.c_uint64, c.c_void_p, c.c_void_p, c.c_void_p]
        _lib.synth_fill_w_fp16.restype = c.c_int
        _lib.synth_fill_w_fp16.argtypes = [c.c_void_p, c.c_int64, c.c_int64, c.c_uint64, c.c_void_p, c.c_void_p]
    return _lib


def _table(device):
    key = str(device)
    if key not in _tables:
        _tables[key] = torch.from_numpy(np.array(G.normal_table())).to(device)
    return _tables[key]


def fill_x(layer, t0=0, t1=None, device="cuda", out=None):
    """X[t0:t1, :] of `layer` as a bf16 CUDA tensor."""
    lib = _load()
    t1 = layer.n_tokens if t1 is None else t1
    n = t1 - t0
    X = torch.empty((n, layer.C), dtype=torch.bfloat16, device=device) if out is None else out
    scales = torch.from_numpy(layer.scales()).to(X.device)
    err = lib.synth_fill_x_bf16(X.data_ptr(), n, layer.C, t0, layer.seed(G.TENSOR_X), _table(X.device).data_ptr(),
                                scales.data_ptr(), ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    if err:
        raise RuntimeError(f"synth_fill_x_bf16: CUDA error {err}")
    torch.cuda.current_stream().synchronize()   # `scales` must outlive the launch
    return X


def fill_w(layer, device="cuda"):
    """W of `layer` as an fp16 CUDA tensor."""
    lib = _load()
    W = torch.empty((layer.R, layer.C), dtype=torch.float16, device=device)
    err = lib.synth_fill_w_fp16(W.data_ptr(), W.numel(), 0, layer.seed(G.TENSOR_W), _table(W.device).data_ptr(),
                                ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    if err:
        raise RuntimeError(f"synth_fill_w_fp16: CUDA error {err}")
    return W

"""The C-ABI library builds, loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2210_17323_b200 import binding_symbols


@pytest.fixture(scope="module")
def lib(repo_root):
    from paper_2210_17323_b200 import build
    path, _ = build.build()
    return ctypes.CDLL(path)


def _declared(repo_root):
    text = open(os.path.join(repo_root, "include", "gptq_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return set(re.findall(r"\b(gptq_[a-z_0-9]+)\s*\(", text))


def test_every_declared_symbol_is_exported(lib, repo_root):
    declared = _declared(repo_root)
    assert declared == set(binding_symbols.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings_and_size_queries_need_no_gpu(lib):
    lib.gptq_status_string.restype = ctypes.c_char_p
    assert lib.gptq_status_string(0) == b"GPTQ_OK"
    assert lib.gptq_status_string(3) == b"GPTQ_ERR_NOT_PD"
    assert lib.gptq_status_string(99) == b"GPTQ_ERR_UNKNOWN"
    lib.gptq_prepare_hinv_workspace_bytes.restype = ctypes.c_size_t
    lib.gptq_quantize_workspace_bytes.restype = ctypes.c_size_t
    assert lib.gptq_prepare_hinv_workspace_bytes(768) % 256 == 0
    small = lib.gptq_quantize_workspace_bytes(768, 768, 4, 0, 128)
    big = lib.gptq_quantize_workspace_bytes(3072, 768, 4, 0, 128)
    assert 0 < small < big
    assert lib.gptq_quantize_workspace_bytes(768, 768, 5, 0, 128) == 0      # unsupported bits

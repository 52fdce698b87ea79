"""The C-ABI library loads without a GPU and exports every declared symbol."""
import ctypes
import os
import re

import pytest

import paper_2504_02692_b200 as g
from paper_2504_02692_b200 import build as gbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    gbuild.build()
    return g.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gptaq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gptaq_[a-zA-Z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_symbols()
    assert len(names) >= 18
    for name in names:
        assert hasattr(lib, name), name
        assert name in g.SIGNATURES, f"{name} has no binding"
    assert sorted(g.SIGNATURES) == names


def test_size_queries_and_host_side_validation(lib):
    n = 128
    sb = g.gptaq_state_bytes(n)
    assert sb >= 2 * n * n * 4 + n and sb % 256 == 0
    assert g.gptaq_state_bytes(0) == 0 and g.gptaq_state_bytes(-3) == 0
    wb = g.gptaq_workspace_bytes(n, 256, 512, 128)
    assert wb >= n * n * 4 + 256 * 2 * 128 * 4
    assert g.gptaq_workspace_bytes(n, 256, 512, 48) == 0          # unsupported block size
    assert g.gptaq_quantize_stage_bytes(8, 128, 0) >= 8 * 128 * 5 + 64
    assert g.gptaq_status_string(g.GPTAQ_ERR_NOT_SPD) == "damped H is not positive definite"
    # null handle / null pointers are rejected on the host, before any CUDA call
    h = ctypes.c_void_p()
    st = lib.gptaq_create(ctypes.byref(h), n, None, sb, None, wb, None)
    assert st == g.GPTAQ_ERR_INVALID_ARG and not h.value
    st = lib.gptaq_create(ctypes.byref(h), n, 256, 16, 512, wb, None)   # state too small
    assert st == g.GPTAQ_ERR_WORKSPACE
    st = lib.gptaq_create(ctypes.byref(h), n, 260, sb, 512, wb, None)   # misaligned
    assert st == g.GPTAQ_ERR_INVALID_ARG
    assert lib.gptaq_factor(None, 0.01, None) == g.GPTAQ_ERR_INVALID_ARG
    assert lib.gptaq_tokens(None) == -1


def test_product_path_has_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        g.LayerState(128, 128, 512, 32)
    # the package never imports the oracle
    import sys
    src = open(os.path.join(ROOT, "paper_2504_02692_b200", "binding.py")).read()
    assert "oracle" not in src.replace("no CPU fallback", "")

"""The C-ABI library builds, loads without a GPU and exports every symbol include/gsa.h declares;
host-side argument checks return error codes without launching anything."""
import ctypes
import os
import re

import pytest

from paper_2601_15305_b200 import binding, build
from paper_2601_15305_b200.inputs import CONFIGS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gsa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gsa_[a-z0-9_]+)\s*\(", text)))


def test_exports_match_header(lib):
    syms = declared_symbols()
    assert "gsa_forward" in syms and "gsa_indexer_scores" in syms and len(syms) >= 10
    for s in syms:
        assert hasattr(lib, s), f"{s} declared in gsa.h but not exported"
    assert set(binding.EXPORTS) <= set(syms)


def test_params_struct_layout_matches_header():
    # 12 int32, 2 float, 3 int32, no padding
    assert ctypes.sizeof(binding.gsa_params_t) == 17 * 4


def test_workspace_bytes_and_argument_errors(lib):
    p = binding.make_params(CONFIGS["l8k"])
    n = binding.gsa_workspace_bytes(p, 0)
    # slab (<= 64 MiB) + V' + idx + kt
    assert n >= 8192 * 4096 * 4 + 8192 * 8 * 128 * 2
    small = binding.gsa_workspace_bytes(p, 32)
    assert small < n
    bad = binding.make_params(CONFIGS["l8k"], d_h=96)
    out = ctypes.c_size_t(0)
    assert lib.gsa_workspace_bytes(ctypes.byref(bad), 0, ctypes.byref(out)) == -2
    bad = binding.make_params(CONFIGS["l8k"], k_min=5000)
    assert lib.gsa_workspace_bytes(ctypes.byref(bad), 0, ctypes.byref(out)) == -1
    assert lib.gsa_workspace_bytes(None, 0, ctypes.byref(out)) == -1
    # NULL tensors are rejected before any CUDA call
    assert lib.gsa_forward(ctypes.byref(p), *([None] * 13), 0, None, ctypes.c_size_t(0), None) == -1
    assert lib.gsa_indexer_scores(ctypes.byref(p), None, None, None, None, None, ctypes.c_int64(8192), None,
                                  ctypes.c_size_t(0), None) == -1
    assert lib.gsa_status_string(-3).decode().startswith("workspace")
    assert binding.gsa_launch_count() == 0

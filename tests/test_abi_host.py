"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol that
include/rmm.h declares, and its host-only logic (keep count, argument validation) behaves."""
import ctypes
import math
import os
import re
from fractions import Fraction

import pytest

from paper_2608_13426_b200 import binding
from paper_2608_13426_b200 import build as rmm_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    rmm_build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "rmm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rmm_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(L):
    names = declared_symbols()
    assert "rmm_score" in names and "rmm_select" in names and "rmm_reduced_gemm" in names and "rmm_reduced_attn" in names
    for n in names:
        assert hasattr(L, n), f"{n} is declared in rmm.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_struct_layouts_match_header(L):
    assert ctypes.sizeof(binding.rmm_mat_t) == 64
    assert ctypes.sizeof(binding.rmm_attn_desc_t) == 6 * 8 + 8 + 16 + 12 * 8 + 8 + 3 * 8


def test_keep_count_host(L):
    for q in (2, 4, 5, 10, 100, 128):
        for p in range(1, q + 1):
            for K in (1, 7, 100, 128, 512, 8192, 28672):
                want = max(1, min(K, math.ceil(Fraction(p, q) * K)))
                assert binding.rmm_keep_count(p / q, K) == want
    for bad in (0.0, -1.0, 1.5, float("nan")):
        with pytest.raises(binding.RmmError) as e:
            binding.rmm_keep_count(bad, 10)
        assert e.value.code == binding.RMM_ERR_INVALID_ARG
    with pytest.raises(binding.RmmError):
        binding.rmm_keep_count(0.5, 0)


def mat(ptr=256, dtype=0, batch=1, rows=4, cols=8, sb=0, sr=8, sc=1):
    return binding.rmm_mat_t(ptr, dtype, batch, rows, cols, sb, sr, sc)


def test_argument_validation_needs_no_gpu(L):
    """Bad arguments are refused on the host before anything is launched."""
    A, B, Y = mat(rows=4, cols=8), mat(rows=8, cols=16, sr=16), mat(rows=4, cols=16, sr=16)
    ws = ctypes.c_void_p(4096)
    # null matrix / null idx
    assert L.rmm_score(None, 1, None, None, ws, 1 << 20, None) == binding.RMM_ERR_INVALID_ARG
    assert L.rmm_reduced_gemm(ctypes.byref(A), ctypes.byref(B), None, 4, 1.0, ctypes.byref(Y), ws, 1 << 20, None) == binding.RMM_ERR_INVALID_ARG
    idx = ctypes.c_void_p(512)
    # k outside [1, K]
    assert L.rmm_reduced_gemm(ctypes.byref(A), ctypes.byref(B), idx, 9, 1.0, ctypes.byref(Y), ws, 1 << 20, None) == binding.RMM_ERR_INVALID_ARG
    assert L.rmm_reduced_gemm(ctypes.byref(A), ctypes.byref(B), idx, 0, 1.0, ctypes.byref(Y), ws, 1 << 20, None) == binding.RMM_ERR_INVALID_ARG
    # inner dimensions disagree
    B2 = mat(rows=9, cols=16, sr=16)
    assert L.rmm_reduced_gemm(ctypes.byref(A), ctypes.byref(B2), idx, 4, 1.0, ctypes.byref(Y), ws, 1 << 20, None) == binding.RMM_ERR_INVALID_ARG
    assert b"columns" in L.rmm_last_error()
    # workspace too small / NULL / misaligned
    assert L.rmm_reduced_gemm(ctypes.byref(A), ctypes.byref(B), idx, 4, 1.0, ctypes.byref(Y), ws, 16, None) == binding.RMM_ERR_WORKSPACE
    assert L.rmm_reduced_gemm(ctypes.byref(A), ctypes.byref(B), idx, 4, 1.0, ctypes.byref(Y), None, 1 << 20, None) == binding.RMM_ERR_WORKSPACE
    assert L.rmm_score_select(ctypes.byref(A), 1, 0.5, 0, idx, None, None, None, ctypes.c_void_p(4100), 1 << 20, None) == binding.RMM_ERR_WORKSPACE
    # rho outside (0, 1]
    assert L.rmm_score_select(ctypes.byref(A), 1, 0.0, 0, idx, None, None, None, ws, 1 << 20, None) == binding.RMM_ERR_INVALID_ARG
    assert L.rmm_score_select(ctypes.byref(A), 1, 1.5, 0, idx, None, None, None, ws, 1 << 20, None) == binding.RMM_ERR_INVALID_ARG
    assert L.rmm_select(ctypes.c_void_p(256), 1, 8, float("nan"), 0, idx, None, ws, 1 << 20, None) == binding.RMM_ERR_INVALID_ARG
    # unknown dtype, bad axis
    assert L.rmm_score(ctypes.byref(mat(dtype=7)), 1, ctypes.c_void_p(256), None, ws, 1 << 20, None) == binding.RMM_ERR_UNSUPPORTED
    assert L.rmm_score(ctypes.byref(A), 2, ctypes.c_void_p(256), None, ws, 1 << 20, None) == binding.RMM_ERR_INVALID_ARG
    # mixed operand dtypes
    assert L.rmm_reduced_gemm(ctypes.byref(A), ctypes.byref(mat(dtype=1, rows=8, cols=16, sr=16)), idx, 4, 1.0, ctypes.byref(Y), ws, 1 << 20, None) == binding.RMM_ERR_UNSUPPORTED


def test_workspace_sizes(L):
    A = mat(rows=2048, cols=8192, sr=8192)
    B = mat(rows=8192, cols=2048, sr=2048)
    Y = mat(rows=2048, cols=2048, sr=2048)
    s = L.rmm_score_select_workspace_bytes(ctypes.byref(A), 1)
    assert s >= 4096 + 8192 * 4
    g = L.rmm_reduced_gemm_workspace_bytes(ctypes.byref(A), ctypes.byref(B), 4096, ctypes.byref(Y))
    assert g >= 4096 + 2048 * 4096 * 2           # packed A[:, I]
    h = L.rmm_product_host_workspace_bytes(2048, 8192, 2048)
    assert h >= g + 2 * 2048 * 8192 * 2 + 2048 * 2048 * 2
    d = binding.rmm_attn_desc_t(1, 4, 2, 128, 128, 64, 1, 0.5, 0.5, (ctypes.c_int64 * 3)(4 * 128 * 64, 128 * 64, 64),
                                (ctypes.c_int64 * 3)(2 * 128 * 64, 128 * 64, 64), (ctypes.c_int64 * 3)(2 * 128 * 64, 128 * 64, 64),
                                (ctypes.c_int64 * 3)(4 * 128 * 64, 128 * 64, 64))
    assert L.rmm_reduced_attn_workspace_bytes(ctypes.byref(d)) > 4096
    d.rho_d = 0.0
    assert L.rmm_reduced_attn_workspace_bytes(ctypes.byref(d)) == 0

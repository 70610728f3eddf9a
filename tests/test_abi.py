"""The C-ABI library builds, loads without a GPU, exports every declared symbol, validates its
arguments on the host, and refuses to compute without a CUDA device (no CPU fallback)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2603_28765_b200 import binding
    binding.lib()
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "abs_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(abs_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(B):
    names = declared_functions()
    assert len(names) >= 12
    L = ctypes.CDLL(B.lib_path())
    for n in names:
        assert hasattr(L, n), f"{n} is declared in include/abs_b200.h but not exported"
    assert sorted(B.EXPORTS) == names


def test_sizes(B):
    assert B.abs_codes_bytes(B.ABS_FMT_IF4, 8192, 4096) == 8192 * 4096 // 2
    assert B.abs_codes_bytes(B.ABS_FMT_NVFP4, 2, 32) == 32
    assert B.abs_codes_bytes(B.ABS_FMT_IF3, 2, 32) == 24
    assert B.abs_codes_bytes(B.ABS_FMT_IF6_E2M3, 2, 32) == 48
    assert B.abs_codes_bytes(B.ABS_FMT_IF6_E3M2, 2, 32) == 48
    assert B.abs_scales_bytes(B.ABS_FMT_IF4, 8192, 4096) == 8192 * 4096 // 16
    assert B.abs_scales_bytes(B.ABS_FMT_IF4_BS8, 8192, 4096) == 8192 * 4096 // 8
    assert B.abs_codes_bytes(B.ABS_FMT_IF4_BS8, 2, 32) == 32 and B.abs_codes_bytes(B.ABS_FMT_IF3_BS8, 2, 32) == 24
    assert B.abs_codes_bytes(B.ABS_FMT_IF4, 2, 30) == 0 and B.abs_codes_bytes(17, 2, 32) == 0
    assert B.abs_codes_bytes(B.ABS_FMT_IF4, -2, 32) == 0
    assert B.abs_host_workspace_bytes(B.ABS_FMT_IF4, 16, 64) >= 16 * 64 * 2 + 16 * 64 // 2 + 64 + 4


def test_status_strings(B):
    seen = {B.status_string(i) for i in range(8)}
    assert len(seen) == 8 and "ok" in seen


def test_alpha_from_amax_is_eq1(B):
    import numpy as np
    assert B.abs_alpha_from_amax(B.ABS_FMT_IF4, 42.0) == 2.0 ** -6
    assert B.abs_alpha_from_amax(B.ABS_FMT_IF4, 0.0) == 1.0
    for fmt, mfp in ((0, 6), (1, 6), (2, 4), (3, 7.5), (4, 28)):
        a = np.float32(3.7)
        assert np.float32(B.abs_alpha_from_amax(fmt, float(a))) == a / np.float32(mfp * 448)


def test_host_side_validation_needs_no_gpu(B):
    L = B.lib()
    dummy = ctypes.c_void_p(0x1000)      # never dereferenced: validation fails first
    assert L.abs_quantize(19, dummy, 4, 64, dummy, dummy, dummy, None) == 4     # format
    assert L.abs_quantize(1, dummy, 4, 60, dummy, dummy, dummy, None) == 2      # cols % 16
    assert L.abs_quantize(1, dummy, -4, 64, dummy, dummy, dummy, None) == 2
    assert L.abs_quantize(1, None, 4, 64, dummy, dummy, dummy, None) == 1       # null
    assert L.abs_quantize(1, ctypes.c_void_p(0x1004), 4, 64, dummy, dummy, dummy, None) == 3   # alignment
    assert L.abs_quantize(1, dummy, 0, 64, dummy, dummy, dummy, None) == 0      # empty: nothing to do
    bad = B.make_opts(1 << 12)
    assert L.abs_quantize_ex(1, dummy, 4, 64, dummy, dummy, dummy, ctypes.byref(bad), None) == 5
    dq = B.make_opts(B.ABS_F_HADAMARD16)
    assert L.abs_dequantize_ex(1, dummy, dummy, dummy, 4, 64, dummy, ctypes.byref(dq), None) == 5
    assert L.abs_dequantize(1, dummy, dummy, dummy, 4, 48 + 8, dummy, None) == 2
    assert L.abs_selftest_convert(7, dummy, 4, dummy, None) == 5


def test_no_cpu_fallback(B):
    """Without a CUDA device a valid call must fail with ABS_ERR_CUDA, never compute on the host."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present; the refusal path is for machines without one")
    L = B.lib()
    dummy = ctypes.c_void_p(0x1000)
    assert L.abs_quantize(1, dummy, 4, 64, dummy, dummy, dummy, None) == 6
    assert L.abs_dequantize(1, dummy, dummy, dummy, 4, 64, dummy, None) == 6
    assert L.abs_init(0) == 6


def test_product_does_not_import_oracle():
    """The CUDA package and the oracle share nothing: neither source tree names the other."""
    pkg = os.path.join(ROOT, "paper_2603_28765_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "abs_oracle" not in text, f
                assert not re.search(r"(?m)^\s*(from|import)\s+oracle\b", text), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c", ".h")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2603_28765_b200" not in text and "abs_b200" not in text, f

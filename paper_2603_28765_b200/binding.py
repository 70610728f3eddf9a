"""Thin ctypes binding of ``libabs_b200.so`` (the C ABI declared in ``include/abs_b200.h``).

Argument marshalling only: every step of quantize / dequantize runs in the library's CUDA
kernels.  PyTorch supplies device memory and streams.  There is no CPU fallback -- if the
library cannot be loaded, or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
import threading

from . import build as _build

(ABS_FMT_NVFP4, ABS_FMT_IF4, ABS_FMT_IF3, ABS_FMT_IF6_E2M3, ABS_FMT_IF6_E3M2, ABS_FMT_NVFP4_BS8, ABS_FMT_IF4_BS8,
 ABS_FMT_IF3_BS8) = range(8)
FMT_NAMES = {"nvfp4": 0, "if4": 1, "if3": 2, "if6_e2m3": 3, "if6_e3m2": 4, "nvfp4_bs8": 5, "if4_bs8": 6, "if3_bs8": 7}
FMT_BITS = {0: 4, 1: 4, 2: 3, 3: 6, 4: 6, 5: 4, 6: 4, 7: 3}
FMT_GROUP = {0: 16, 1: 16, 2: 16, 3: 16, 4: 16, 5: 8, 6: 8, 7: 8}

ABS_F_HADAMARD16 = 1 << 0
ABS_F_STOCHASTIC = 1 << 1
ABS_F_SR_SCALE_17_16 = 1 << 2
ABS_F_ALPHA_GIVEN = 1 << 3
ABS_F_OUT_FP32 = 1 << 4
ABS_F_INDEX64 = 1 << 5
ABS_F_SCALES_SWIZZLED = 1 << 6
ABS_F_GROUPS_DOWN_COLUMNS = 1 << 9
ABS_F_FP_GROUPS_ONLY = 1 << 7
ABS_F_INT_GROUPS_RAW = 1 << 8

ABS_OK = 0

EXPORTS = [
    "abs_codes_bytes", "abs_scales_bytes", "abs_status_string", "abs_init", "abs_quantize", "abs_quantize_ex",
    "abs_dequantize", "abs_dequantize_ex", "abs_amax", "abs_alpha_from_amax", "abs_host_workspace_bytes",
    "abs_quantize_host", "abs_dequantize_host", "abs_selftest_convert", "abs_profile_events",
    "abs_quantize_noalloc", "abs_quantize_transposed", "abs_scales_bytes_swizzled", "abs_quantize_dequantize",
    "abs_matmul_workspace_bytes", "abs_matmul", "abs_matmul_bf16", "abs_matmul_bf16_scaled", "abs_matmul_check",
    "abs_selftest_matmul_stall",
]


class AbsOpts(C.Structure):
    _fields_ = [("flags", C.c_uint32), ("had_sign_mask", C.c_uint16), ("_pad", C.c_uint16), ("sr_seed", C.c_uint64),
                ("sr_index_offset", C.c_uint64)]


class AbsError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: status {status} ({status_string(status)})")
        self.status = status


_lock = threading.Lock()
_lib = None


def lib_path() -> str:
    return _build.LIB_PATH


def lib():
    """Loads (building first if the sources are newer) the CUDA library. Raises if unavailable."""
    global _lib
    with _lock:
        if _lib is None:
            path = _build.LIB_PATH
            if not os.path.exists(path) or _build.needs_build():
                path = _build.build()
            L = C.CDLL(path)
            vp, i64, sz = C.c_void_p, C.c_int64, C.c_size_t
            op = C.POINTER(AbsOpts)
            L.abs_codes_bytes.restype = sz
            L.abs_codes_bytes.argtypes = [C.c_int, i64, i64]
            L.abs_scales_bytes.restype = sz
            L.abs_scales_bytes.argtypes = [C.c_int, i64, i64]
            L.abs_scales_bytes_swizzled.restype = sz
            L.abs_scales_bytes_swizzled.argtypes = [C.c_int, i64, i64]
            L.abs_status_string.restype = C.c_char_p
            L.abs_status_string.argtypes = [C.c_int]
            L.abs_init.restype = C.c_int
            L.abs_init.argtypes = [C.c_int]
            L.abs_quantize.restype = C.c_int
            L.abs_quantize.argtypes = [C.c_int, vp, i64, i64, vp, vp, vp, vp]
            L.abs_quantize_ex.restype = C.c_int
            L.abs_quantize_ex.argtypes = [C.c_int, vp, i64, i64, vp, vp, vp, op, vp]
            L.abs_quantize_transposed.restype = C.c_int
            L.abs_quantize_transposed.argtypes = [C.c_int, vp, i64, i64, vp, vp, vp, op, vp]
            L.abs_quantize_dequantize.restype = C.c_int
            L.abs_quantize_dequantize.argtypes = [C.c_int, vp, i64, i64, vp, vp, vp, vp, op, vp]
            L.abs_quantize_noalloc.restype = C.c_int
            L.abs_quantize_noalloc.argtypes = [C.c_int, vp, i64, i64, vp, vp, vp, vp]
            L.abs_dequantize.restype = C.c_int
            L.abs_dequantize.argtypes = [C.c_int, vp, vp, vp, i64, i64, vp, vp]
            L.abs_dequantize_ex.restype = C.c_int
            L.abs_dequantize_ex.argtypes = [C.c_int, vp, vp, vp, i64, i64, vp, op, vp]
            L.abs_amax.restype = C.c_int
            L.abs_amax.argtypes = [vp, i64, i64, op, vp, vp]
            L.abs_alpha_from_amax.restype = C.c_float
            L.abs_alpha_from_amax.argtypes = [C.c_int, C.c_float]
            L.abs_host_workspace_bytes.restype = sz
            L.abs_host_workspace_bytes.argtypes = [C.c_int, i64, i64]
            L.abs_quantize_host.restype = C.c_int
            L.abs_quantize_host.argtypes = [C.c_int, vp, i64, i64, vp, vp, vp, op, vp, sz, vp]
            L.abs_dequantize_host.restype = C.c_int
            L.abs_dequantize_host.argtypes = [C.c_int, vp, vp, vp, i64, i64, vp, op, vp, sz, vp]
            L.abs_matmul_workspace_bytes.restype = sz
            L.abs_matmul_workspace_bytes.argtypes = [C.c_int, i64, i64, i64]
            L.abs_matmul.restype = C.c_int
            L.abs_matmul.argtypes = [C.c_int, vp, vp, vp, vp, vp, vp, i64, i64, i64, vp, vp, sz, vp]
            L.abs_matmul_bf16.restype = C.c_int
            L.abs_matmul_bf16.argtypes = [C.c_int, vp, vp, vp, vp, vp, vp, i64, i64, i64, vp, vp, sz, vp]
            L.abs_matmul_bf16_scaled.restype = C.c_int
            L.abs_matmul_bf16_scaled.argtypes = [C.c_int, vp, vp, vp, vp, vp, vp, i64, i64, i64, vp, C.c_int, vp, vp, sz, vp]
            L.abs_matmul_check.restype = C.c_int
            L.abs_matmul_check.argtypes = [vp, vp]
            L.abs_selftest_matmul_stall.restype = C.c_int
            L.abs_selftest_matmul_stall.argtypes = [C.c_int, vp, vp, vp, vp, vp, vp, i64, i64, i64, vp, vp, sz, vp, C.c_int32]
            L.abs_profile_events.restype = None
            L.abs_profile_events.argtypes = [vp, vp]
            L.abs_selftest_convert.restype = C.c_int
            L.abs_selftest_convert.argtypes = [C.c_int, vp, i64, vp, vp]
            _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().abs_status_string(status).decode()


def _check(status: int, what: str):
    if status != ABS_OK:
        raise AbsError(status, what)


def make_opts(flags: int = 0, had_sign_mask: int = 0, sr_seed: int = 0, sr_index_offset: int = 0) -> AbsOpts:
    return AbsOpts(flags, had_sign_mask, 0, sr_seed, sr_index_offset)


def _stream_ptr(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def abs_codes_bytes(fmt: int, rows: int, cols: int) -> int:
    return lib().abs_codes_bytes(fmt, rows, cols)


def abs_scales_bytes(fmt: int, rows: int, cols: int) -> int:
    return lib().abs_scales_bytes(fmt, rows, cols)


def abs_scales_bytes_swizzled(fmt: int, rows: int, cols: int) -> int:
    return lib().abs_scales_bytes_swizzled(fmt, rows, cols)


def abs_alpha_from_amax(fmt: int, amax: float) -> float:
    return lib().abs_alpha_from_amax(fmt, amax)


def abs_init(device: int = 0):
    _check(lib().abs_init(device), "abs_init")


def abs_quantize(fmt: int, x, codes=None, scales=None, tensor_scale=None, opts: AbsOpts | None = None, stream=None):
    """Quantize a CUDA bf16 matrix ``x`` [rows, cols] (contiguous).

    Output buffers are allocated with torch when not given.  Returns (codes u8, scales u8,
    tensor_scale f32[1]); with ABS_F_ALPHA_GIVEN ``tensor_scale`` is the input alpha."""
    import torch
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.is_contiguous()
    rows, cols = x.shape
    L = lib()
    if codes is None:
        codes = torch.empty(max(L.abs_codes_bytes(fmt, rows, cols), 1) if cols % 16 == 0 else 1, dtype=torch.uint8,
                            device=x.device)
    if scales is None:
        if opts is not None and (opts.flags & ABS_F_SCALES_SWIZZLED):
            scales = torch.zeros(max(L.abs_scales_bytes_swizzled(fmt, rows, cols), 1), dtype=torch.uint8, device=x.device)
        else:
            scales = torch.empty(max(rows * cols // FMT_GROUP[fmt], 1), dtype=torch.uint8, device=x.device)
    if tensor_scale is None:
        tensor_scale = torch.zeros(1, dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        rc = L.abs_quantize_ex(fmt, x.data_ptr(), rows, cols, codes.data_ptr(), scales.data_ptr(),
                               tensor_scale.data_ptr(), C.byref(opts) if opts is not None else None,
                               _stream_ptr(stream))
    _check(rc, "abs_quantize")
    return codes, scales, tensor_scale


def abs_quantize_transposed(fmt: int, x, codes_t=None, scales_t=None, tensor_scale=None, opts: AbsOpts | None = None,
                            stream=None):
    """Quantize the transpose of the CUDA bf16 matrix ``x`` [rows, cols] (groups of 16 down the columns)
    without materialising it.  Returns (codes_t u8 [cols*rows*b/8], scales_t u8 [cols*rows/16], alpha)."""
    import torch
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.is_contiguous()
    rows, cols = x.shape
    if codes_t is None:
        codes_t = torch.empty(max(rows * cols * FMT_BITS[fmt] // 8, 1), dtype=torch.uint8, device=x.device)
    if scales_t is None:
        scales_t = torch.empty(max(rows * cols // 16, 1), dtype=torch.uint8, device=x.device)
    if tensor_scale is None:
        tensor_scale = torch.zeros(1, dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        rc = lib().abs_quantize_transposed(fmt, x.data_ptr(), rows, cols, codes_t.data_ptr(), scales_t.data_ptr(),
                                           tensor_scale.data_ptr(), C.byref(opts) if opts is not None else None,
                                           _stream_ptr(stream))
    _check(rc, "abs_quantize_transposed")
    return codes_t, scales_t, tensor_scale


def abs_quantize_dequantize(fmt: int, x, out=None, codes=None, scales=None, tensor_scale=None,
                            opts: AbsOpts | None = None, stream=None):
    """Quantize the CUDA bf16 matrix ``x`` and dequantize it in the same pass (the emulation of Sec. 4.1).
    ``codes`` and ``scales`` are optional outputs (both or neither).  Returns (out bf16 [rows, cols], alpha)."""
    import torch
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.is_contiguous()
    rows, cols = x.shape
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.bfloat16, device=x.device)
    if tensor_scale is None:
        tensor_scale = torch.zeros(1, dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        rc = lib().abs_quantize_dequantize(fmt, x.data_ptr(), rows, cols, out.data_ptr(),
                                           codes.data_ptr() if codes is not None else None,
                                           scales.data_ptr() if scales is not None else None, tensor_scale.data_ptr(),
                                           C.byref(opts) if opts is not None else None, _stream_ptr(stream))
    _check(rc, "abs_quantize_dequantize")
    return out, tensor_scale


def abs_quantize_noalloc(fmt: int, x, codes, scales, tensor_scale, stream=None):
    """Quantize with the variant of the library that allocates nothing (see ``abs_quantize_noalloc`` in
    the header): for processes that cannot call cudaMalloc any more.  All buffers come from the caller,
    so nothing is allocated here either; at most 2**30 elements; do not overlap two calls on one GPU."""
    import torch
    rows, cols = x.shape
    with torch.cuda.device(x.device):
        rc = lib().abs_quantize_noalloc(fmt, x.data_ptr(), rows, cols, codes.data_ptr(), scales.data_ptr(),
                                        tensor_scale.data_ptr(), _stream_ptr(stream))
    _check(rc, "abs_quantize_noalloc")
    return codes, scales, tensor_scale


def abs_dequantize(fmt: int, codes, scales, tensor_scale, rows: int, cols: int, out=None,
                   opts: AbsOpts | None = None, stream=None):
    """Dequantize to a CUDA bf16 matrix (float32 with ABS_F_OUT_FP32)."""
    import torch
    fp32 = bool(opts is not None and (opts.flags & ABS_F_OUT_FP32))
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.float32 if fp32 else torch.bfloat16, device=codes.device)
    with torch.cuda.device(codes.device):
        rc = lib().abs_dequantize_ex(fmt, codes.data_ptr(), scales.data_ptr(), tensor_scale.data_ptr(), rows, cols,
                                     out.data_ptr(), C.byref(opts) if opts is not None else None, _stream_ptr(stream))
    _check(rc, "abs_dequantize")
    return out


def abs_matmul(fmt: int, qa, qb, m: int, n: int, k: int, out=None, workspace=None, stream=None, check: bool = False,
               bf16: bool = False, next_fmt: int | None = None, next_alpha=None):
    """C = A B^T on the tensor cores for two quantized operands ``qa`` = (codes, scales, alpha) of A [m, k] and
    ``qb`` of B [n, k] (row-major scales), with the MAC arithmetic of Sec. 5.2.  Returns C as float32 [m, n], or with
    ``bf16`` as bfloat16 (the same values rounded to nearest even).  With ``next_fmt`` (bf16 output only) the kernel also
    leaves the tensor scale that ``abs_quantize(next_fmt, C)`` would compute in ``next_alpha`` (a CUDA float32[1],
    allocated when not given) and the call returns (C, next_alpha).  ``check`` synchronises and raises if a wait inside
    the kernel ran out."""
    import torch
    L = lib()
    need = L.abs_matmul_workspace_bytes(fmt, m, n, k)
    if need == 0:
        raise AbsError(2, "abs_matmul: n a multiple of 128 and k a multiple of 256; IF4 or NVFP4")
    if workspace is None:
        workspace = torch.empty(need + 1024, dtype=torch.uint8, device=qa[0].device)
    off = (-workspace.data_ptr()) % 1024
    if out is None:
        out = torch.empty((m, n), dtype=torch.bfloat16 if bf16 else torch.float32, device=qa[0].device)
    assert out.dtype == (torch.bfloat16 if bf16 else torch.float32)
    with torch.cuda.device(qa[0].device):
        sp = _stream_ptr(stream)
        if next_fmt is not None:
            assert bf16
            if next_alpha is None:
                next_alpha = torch.zeros(1, dtype=torch.float32, device=qa[0].device)
            rc = L.abs_matmul_bf16_scaled(fmt, qa[0].data_ptr(), qa[1].data_ptr(), qa[2].data_ptr(), qb[0].data_ptr(),
                                          qb[1].data_ptr(), qb[2].data_ptr(), m, n, k, out.data_ptr(), next_fmt,
                                          next_alpha.data_ptr(), workspace.data_ptr() + off, workspace.numel() - off, sp)
            _check(rc, "abs_matmul_bf16_scaled")
            if check:
                _check(L.abs_matmul_check(workspace.data_ptr() + off, sp), "abs_matmul (a wait inside the kernel ran out)")
            return out, next_alpha
        rc = (L.abs_matmul_bf16 if bf16 else L.abs_matmul)(fmt, qa[0].data_ptr(), qa[1].data_ptr(), qa[2].data_ptr(), qb[0].data_ptr(), qb[1].data_ptr(),
                          qb[2].data_ptr(), m, n, k, out.data_ptr(), workspace.data_ptr() + off, workspace.numel() - off, sp)
        _check(rc, "abs_matmul")
        if check:
            _check(L.abs_matmul_check(workspace.data_ptr() + off, sp), "abs_matmul (a wait inside the kernel ran out)")
    return out


def abs_amax(x, opts: AbsOpts | None = None, out=None, stream=None):
    """Grid-wide max |x| (after the Hadamard option when asked) into a CUDA float32[1]."""
    import torch
    rows, cols = x.shape
    if out is None:
        out = torch.zeros(1, dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        rc = lib().abs_amax(x.data_ptr(), rows, cols, C.byref(opts) if opts is not None else None, out.data_ptr(),
                            _stream_ptr(stream))
    _check(rc, "abs_amax")
    return out


def abs_host_workspace_bytes(fmt: int, rows: int, cols: int) -> int:
    return lib().abs_host_workspace_bytes(fmt, rows, cols)


def abs_quantize_host(fmt: int, x_host, codes_host, scales_host, alpha_host, workspace, opts: AbsOpts | None = None,
                      stream=None):
    """Host-buffer variant: ``*_host`` are CPU tensors (pinned for speed), ``workspace`` a CUDA u8 tensor."""
    rows, cols = x_host.shape
    import torch
    with torch.cuda.device(workspace.device):
        rc = lib().abs_quantize_host(fmt, x_host.data_ptr(), rows, cols, codes_host.data_ptr(), scales_host.data_ptr(),
                                     alpha_host.data_ptr(), C.byref(opts) if opts is not None else None,
                                     workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _check(rc, "abs_quantize_host")


def abs_dequantize_host(fmt: int, codes_host, scales_host, alpha_host, rows: int, cols: int, out_host, workspace,
                        opts: AbsOpts | None = None, stream=None):
    import torch
    with torch.cuda.device(workspace.device):
        rc = lib().abs_dequantize_host(fmt, codes_host.data_ptr(), scales_host.data_ptr(), alpha_host.data_ptr(), rows,
                                       cols, out_host.data_ptr(), C.byref(opts) if opts is not None else None,
                                       workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _check(rc, "abs_dequantize_host")


def abs_profile_events(begin_event=None, end_event=None):
    """Records the two torch CUDA events around the group-quantize kernel of later quantize calls;
    call with no arguments to switch the hook off."""
    lib().abs_profile_events(C.c_void_p(begin_event.cuda_event) if begin_event is not None else None,
                             C.c_void_p(end_event.cuda_event) if end_event is not None else None)


def abs_selftest_convert(kind: int, x_f32, out=None, stream=None):
    import torch
    n = x_f32.numel()
    if out is None:
        out = torch.empty(n, dtype=torch.uint8 if kind < 16 else torch.float32, device=x_f32.device)
    with torch.cuda.device(x_f32.device):
        rc = lib().abs_selftest_convert(kind, x_f32.data_ptr(), n, out.data_ptr(), _stream_ptr(stream))
    _check(rc, "abs_selftest_convert")
    return out

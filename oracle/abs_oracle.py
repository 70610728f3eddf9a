"""ctypes front end of the CPU oracle (``abs_oracle.c``).

TEST INFRASTRUCTURE, NOT PRODUCT: only the tests, the smoke check and the bench's
``cpu_baseline`` / reference arm import this module.  It never imports the CUDA package.

All the method's arithmetic lives in the C file; this module only builds it with gcc,
marshals numpy arrays, and (for timing) splits rows over Python threads -- ctypes releases
the GIL during a foreign call, so the row chunks run on separate host cores.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "abs_oracle.c")
_LIB = os.path.join(_HERE, "libabs_oracle.so")

FMT_NVFP4, FMT_IF4, FMT_IF3, FMT_IF6_E2M3, FMT_IF6_E3M2, FMT_NVFP4_BS8, FMT_IF4_BS8, FMT_IF3_BS8 = range(8)
FMT_NAMES = {"nvfp4": 0, "if4": 1, "if3": 2, "if6_e2m3": 3, "if6_e3m2": 4, "nvfp4_bs8": 5, "if4_bs8": 6, "if3_bs8": 7}

F_HADAMARD16 = 1 << 0
F_STOCHASTIC = 1 << 1
F_SR_SCALE_17_16 = 1 << 2
F_ALPHA_GIVEN = 1 << 3
F_OUT_FP32 = 1 << 4
F_FP_GROUPS_ONLY = 1 << 7
F_INT_GROUPS_RAW = 1 << 8

_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (plain C, no contraction, no fast-math). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fvisibility=hidden",
               "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            u8p, u16p, f32p, u32p = (C.POINTER(t) for t in (C.c_uint8, C.c_uint16, C.c_float, C.c_uint32))
            L.abs_oracle_fmt_bits.restype = C.c_int
            L.abs_oracle_fmt_bits.argtypes = [C.c_int]
            L.abs_oracle_fmt_group.restype = C.c_int
            L.abs_oracle_fmt_group.argtypes = [C.c_int]
            for name in ("abs_oracle_fmt_mfp", "abs_oracle_fmt_mint", "abs_oracle_c_pre", "abs_oracle_c_post"):
                getattr(L, name).restype = C.c_float
                getattr(L, name).argtypes = [C.c_int]
            L.abs_oracle_fp_value.restype = C.c_float
            L.abs_oracle_fp_value.argtypes = [C.c_int, C.c_uint32]
            L.abs_oracle_fp_encode.restype = C.c_uint32
            L.abs_oracle_fp_encode.argtypes = [C.c_int, C.c_float]
            L.abs_oracle_int_encode.restype = C.c_int
            L.abs_oracle_int_encode.argtypes = [C.c_int, C.c_float]
            L.abs_oracle_e4m3_encode.restype = C.c_uint32
            L.abs_oracle_e4m3_encode.argtypes = [C.c_float]
            L.abs_oracle_e4m3_value.restype = C.c_float
            L.abs_oracle_e4m3_value.argtypes = [C.c_uint32]
            L.abs_oracle_philox4x32_10.restype = None
            L.abs_oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
            L.abs_oracle_sr_uniform.restype = C.c_float
            L.abs_oracle_sr_uniform.argtypes = [C.c_uint64, C.c_uint64]
            L.abs_oracle_fp_sr.restype = C.c_int
            L.abs_oracle_fp_sr.argtypes = [C.c_int, C.c_float, C.c_float]
            L.abs_oracle_hadamard16.restype = None
            L.abs_oracle_hadamard16.argtypes = [f32p, C.c_uint16, f32p]
            L.abs_oracle_f32_to_bf16.restype = C.c_uint16
            L.abs_oracle_f32_to_bf16.argtypes = [C.c_float]
            L.abs_oracle_amax.restype = C.c_float
            L.abs_oracle_amax.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_uint32, C.c_uint16]
            L.abs_oracle_alpha.restype = C.c_float
            L.abs_oracle_alpha.argtypes = [C.c_int, C.c_float]
            L.abs_oracle_quantize_rows.restype = C.c_int
            L.abs_oracle_quantize_rows.argtypes = [C.c_int, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int64,
                                                   C.c_float, C.c_uint32, C.c_uint16, C.c_uint64, C.c_uint64,
                                                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
            L.abs_oracle_dequantize_rows.restype = C.c_int
            L.abs_oracle_dequantize_rows.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_float, C.c_int64,
                                                     C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_void_p, C.c_uint32]
            _lib = L
    return _lib


# ----------------------------------------------------------------------------- scalar pieces

def fmt_bits(fmt: int) -> int:
    return lib().abs_oracle_fmt_bits(fmt)


def fmt_group(fmt: int) -> int:
    """Values that share one scale: 16, or 8 for the block-size-8 variants."""
    return lib().abs_oracle_fmt_group(fmt)


def codes_bytes(fmt: int, rows: int, cols: int) -> int:
    return rows * cols * fmt_bits(fmt) // 8


def scales_bytes(rows: int, cols: int, fmt: int = 0) -> int:
    return rows * cols // fmt_group(fmt)


def c_pre(fmt):
    return np.float32(lib().abs_oracle_c_pre(fmt))


def c_post(fmt):
    return np.float32(lib().abs_oracle_c_post(fmt))


def m_fp(fmt):
    return np.float32(lib().abs_oracle_fmt_mfp(fmt))


def m_int(fmt):
    return np.float32(lib().abs_oracle_fmt_mint(fmt))


def fp_value(fmt: int, code: int) -> np.float32:
    return np.float32(lib().abs_oracle_fp_value(fmt, code))


def fp_encode(fmt: int, y) -> int:
    return int(lib().abs_oracle_fp_encode(fmt, C.c_float(float(np.float32(y)))))


def int_encode(fmt: int, y) -> int:
    return int(lib().abs_oracle_int_encode(fmt, C.c_float(float(np.float32(y)))))


def e4m3_encode(t) -> int:
    return int(lib().abs_oracle_e4m3_encode(C.c_float(float(np.float32(t)))))


def e4m3_value(byte: int) -> np.float32:
    return np.float32(lib().abs_oracle_e4m3_value(byte))


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().abs_oracle_philox4x32_10(c, k, o)
    return [int(v) for v in o]


def sr_uniform(seed: int, idx: int) -> np.float32:
    return np.float32(lib().abs_oracle_sr_uniform(seed, idx))


def fp_sr(fmt: int, a: float, u: float) -> int:
    """Index on the FP grid of ``fmt`` that the magnitude ``a`` rounds to stochastically for the uniform ``u``."""
    return int(lib().abs_oracle_fp_sr(fmt, float(a), float(u)))


def hadamard16(x16, sign_mask: int) -> np.ndarray:
    a = np.ascontiguousarray(x16, dtype=np.float32)
    assert a.shape == (16,)
    o = np.empty(16, dtype=np.float32)
    f32p = C.POINTER(C.c_float)
    lib().abs_oracle_hadamard16(a.ctypes.data_as(f32p), sign_mask, o.ctypes.data_as(f32p))
    return o


def f32_to_bf16(f) -> int:
    return int(lib().abs_oracle_f32_to_bf16(C.c_float(float(np.float32(f)))))


def hadamard_sign_mask(seed: int) -> int:
    """Sign vector of the Hadamard option derived from a seed: low 16 bits of word 0 of
    Philox4x32-10(counter = (0, 0, 1, 0), key = seed)."""
    w = philox4x32_10([0, 0, 1, 0], [seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF])
    return w[0] & 0xFFFF


# ----------------------------------------------------------------------------- tensor level

def _chunks(rows: int, threads: int):
    threads = max(1, min(threads, rows))
    edges = [rows * i // threads for i in range(threads + 1)]
    return [(edges[i], edges[i + 1]) for i in range(threads) if edges[i + 1] > edges[i]]


def _as_u16(x_bf16_bits) -> np.ndarray:
    a = np.ascontiguousarray(x_bf16_bits)
    assert a.dtype == np.uint16 and a.ndim == 2, "input is a 2-D array of bf16 bit patterns (uint16)"
    return a


def amax(x_bf16_bits, flags: int = 0, sign_mask: int = 0, threads: int = 1) -> np.float32:
    a = _as_u16(x_bf16_bits)
    rows, cols = a.shape
    assert cols % 16 == 0
    L = lib()
    if rows * cols == 0:
        return np.float32(0.0)

    def work(rr):
        return L.abs_oracle_amax(a.ctypes.data, cols, rr[0], rr[1], flags, sign_mask)

    if threads <= 1:
        return np.float32(work((0, rows)))
    with ThreadPoolExecutor(threads) as ex:
        return np.float32(max(ex.map(work, _chunks(rows, threads))))


def alpha_from_amax(fmt: int, A) -> np.float32:
    return np.float32(lib().abs_oracle_alpha(fmt, C.c_float(float(A))))


def quantize(fmt: int, x_bf16_bits, flags: int = 0, sign_mask: int = 0, sr_seed: int = 0,
             alpha=None, threads: int = 1, debug: bool = False, sr_index_offset: int = 0):
    """Quantize a 2-D array of bf16 bit patterns.  ``sr_index_offset``: index of element (0, 0) in the
    whole tensor when the array is a row shard of a larger one (stochastic rounding only).

    Returns (codes u8[rows, cols*b/8], scales u8[rows, cols/16], alpha float32) and, with
    ``debug``, additionally (E_FP, E_INT) per group as float32[rows, cols/16]."""
    a = _as_u16(x_bf16_bits)
    rows, cols = a.shape
    assert cols % 16 == 0
    b = fmt_bits(fmt)
    L = lib()
    if flags & F_ALPHA_GIVEN:
        assert alpha is not None
        alpha = np.float32(alpha)
    else:
        alpha = alpha_from_amax(fmt, amax(a, flags, sign_mask, threads))
    G = fmt_group(fmt)
    codes = np.zeros((rows, cols * b // 8), dtype=np.uint8)
    scales = np.zeros((rows, cols // G), dtype=np.uint8)
    efp = np.zeros((rows, cols // G), dtype=np.float32) if debug else None
    eint = np.zeros((rows, cols // G), dtype=np.float32) if debug else None

    def work(rr):
        rc = L.abs_oracle_quantize_rows(fmt, a.ctypes.data, rows, cols, rr[0], rr[1], C.c_float(float(alpha)),
                                        flags, sign_mask, sr_seed, sr_index_offset, codes.ctypes.data,
                                        scales.ctypes.data,
                                        efp.ctypes.data if debug else None, eint.ctypes.data if debug else None)
        if rc != 0:
            raise ValueError("abs_oracle_quantize_rows rejected its arguments")

    if rows * cols:
        if threads <= 1:
            work((0, rows))
        else:
            with ThreadPoolExecutor(threads) as ex:
                list(ex.map(work, _chunks(rows, threads)))
    if debug:
        return codes, scales, alpha, efp, eint
    return codes, scales, alpha


def dequantize(fmt: int, codes, scales, alpha, rows: int, cols: int, out_fp32: bool = False, threads: int = 1,
               select: int = 0):
    """Inverse path. Returns bf16 bit patterns (uint16) or float32 when ``out_fp32``.  ``select`` =
    F_FP_GROUPS_ONLY or F_INT_GROUPS_RAW gives one half of the split used for the MAC arithmetic."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    assert codes.size == codes_bytes(fmt, rows, cols) and scales.size == scales_bytes(rows, cols, fmt)
    out = np.zeros((rows, cols), dtype=np.float32 if out_fp32 else np.uint16)
    L = lib()

    def work(rr):
        rc = L.abs_oracle_dequantize_rows(fmt, codes.ctypes.data, scales.ctypes.data, C.c_float(float(alpha)),
                                          rows, cols, rr[0], rr[1], int(out_fp32), out.ctypes.data, select)
        if rc != 0:
            raise ValueError("abs_oracle_dequantize_rows rejected its arguments")

    if rows * cols:
        if threads <= 1:
            work((0, rows))
        else:
            with ThreadPoolExecutor(threads) as ex:
                list(ex.map(work, _chunks(rows, threads)))
    return out


def bf16_bits_to_f32(bits) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32 (a dtype view, no rounding)."""
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def swizzle_scales(scales: np.ndarray, fill: int = 0) -> np.ndarray:
    """Row-major scale bytes [rows, K] -> the 128x4-tile layout that Blackwell block-scaled tensor-core
    MMAs read (the layout NVFP4 kernels use for their E4M3 scales; Sec. 3: an FP group IS an NVFP4
    group).  Written as the layout's definition: pad to whole 128 x 4 tiles; tiles in row-major order;
    inside a tile the 128 rows are split as (row // 32, row % 32) and stored with row % 32 slowest,
    then row // 32, then the 4 scales of the row.  Padding bytes get ``fill``."""
    s = np.asarray(scales, dtype=np.uint8)
    rows, k = s.shape
    mt, kt = -(-rows // 128), -(-k // 4)
    padded = np.full((mt * 128, kt * 4), fill, dtype=np.uint8)
    padded[:rows, :k] = s
    tiles = padded.reshape(mt, 4, 32, kt, 4)           # [tile row, row // 32, row % 32, tile col, scale]
    return np.ascontiguousarray(tiles.transpose(0, 3, 2, 1, 4)).reshape(-1)   # [mt, kt, row % 32, row // 32, scale]


def mac_matmul_reference(fmt: int, qa, qb, m: int, n: int, k: int) -> np.ndarray:
    """C = A B^T for two quantized operands (A: [m, k], B: [n, k], groups along k) with the arithmetic of
    the paper's MAC unit (Sec. 5.2), in float64: inside a group pair the decoded codes are multiplied and
    summed exactly; the sum is scaled by Delta_a * Delta_b and by 1, 6/7 or 36/49 when none, one or both
    groups are integer groups; the tensor scales multiply the total.  qa, qb = (codes, scales, alpha)."""
    parts = []
    for codes, scales, alpha, rows in ((qa[0], qa[1], qa[2], m), (qb[0], qb[1], qb[2], n)):
        fp = dequantize(fmt, codes, scales, 1.0, rows, k, out_fp32=True, select=F_FP_GROUPS_ONLY).astype(np.float64)
        it = dequantize(fmt, codes, scales, 1.0, rows, k, out_fp32=True, select=F_INT_GROUPS_RAW).astype(np.float64)
        parts.append((fp, it, float(alpha)))
    (af, ai, aa), (bf, bi, ab) = parts
    if float(m_int(fmt)) == 0.0:                      # plain NVFP4: there are no integer groups
        return (af @ bf.T) * (aa * ab)
    c67 = float(m_fp(fmt)) / float(m_int(fmt))
    c = af @ bf.T + c67 * (af @ bi.T + ai @ bf.T) + (c67 * c67) * (ai @ bi.T)
    return c * (aa * ab)

"""Seeded synthetic inputs shared by the oracle tests, the GPU tests and the bench.

This module holds no arithmetic of the method: it only draws random tensors with the
shapes and value distributions of the benchmark configurations and converts them to bf16
bit patterns (uint16).  The same bytes are handed to the CPU oracle and to the CUDA path.

They stand in for the tensors the paper quantizes (model weights, activations and
gradients, Sec. 4), which need trained models and datasets.

Recipe (numpy ``Generator(PCG64(seed))``, draws in the order written, float32 unless noted):
  cfg1  256 x 1024      N(0,1), seed 0
  cfg2  8192 x 4096     0.5 * Student-t(df=3) (float64 draw), then 0.5 % of the columns
                        (``rng.choice`` without replacement, drawn first) multiplied by 50
  cfg3a 4096 x 14336    N(0, 0.02^2), seed 3
  cfg3b 14336 x 4096    N(0, 0.02^2), seed 4
  cfg4  16384 x 8192    per-row magnitude 10^U(-2,2) (drawn first, float64) times N(0,(1e-3)^2)
  cfg5  16384 x 8192    per element: N(0,1) w.p. 0.7 else Laplace(0,1); then x100 w.p. 0.001
                        (draw order per row block: selector uniform, normal, laplace, outlier uniform)
Rows are generated in blocks of 1024 so memory stays bounded; a smaller ``rows`` simply
stops early, so a reduced-size tensor is a prefix of the full one.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass

import numpy as np

_BLOCK = 1024


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns, round to nearest even (inputs are finite)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class Config:
    name: str
    rows: int
    cols: int
    seed: int
    kind: str
    note: str


CONFIGS = {
    "cfg1": Config("cfg1", 256, 1024, 0, "normal", "N(0,1)"),
    "cfg2": Config("cfg2", 8192, 4096, 2, "activation", "0.5*t(3), 0.5% outlier columns x50"),
    "cfg3a": Config("cfg3a", 4096, 14336, 3, "weight", "N(0,0.02^2)"),
    "cfg3b": Config("cfg3b", 14336, 4096, 4, "weight", "N(0,0.02^2)"),
    "cfg4": Config("cfg4", 16384, 8192, 5, "gradient", "N(0,1e-6) x per-row 10^U(-2,2)"),
    "cfg5": Config("cfg5", 16384, 8192, 6, "mixture", "0.7 N(0,1) + 0.3 Laplace(0,1), 0.1% x100"),
}


def _blocks(rows: int):
    r = 0
    while r < rows:
        n = min(_BLOCK, rows - r)
        yield r, n
        r += n


def generate(name: str, rows: int | None = None, cols: int | None = None, seed: int | None = None) -> np.ndarray:
    """bf16 bit patterns (uint16, shape [rows, cols]) of configuration ``name``.

    ``rows`` / ``cols`` / ``seed`` override the configuration's values (reduced-size cases)."""
    cfg = CONFIGS[name]
    rows = cfg.rows if rows is None else rows
    cols = cfg.cols if cols is None else cols
    seed = cfg.seed if seed is None else seed
    rng = np.random.Generator(np.random.PCG64(seed))
    out = np.empty((rows, cols), dtype=np.uint16)
    if cfg.kind == "normal":
        for r, n in _blocks(rows):
            out[r:r + n] = f32_to_bf16_bits(rng.standard_normal((n, cols), dtype=np.float32))
    elif cfg.kind == "activation":
        k = max(1, int(round(0.005 * cols)))
        hot = rng.choice(cols, size=k, replace=False)
        colscale = np.ones(cols, dtype=np.float32)
        colscale[hot] = 50.0
        for r, n in _blocks(rows):
            t = (0.5 * rng.standard_t(3.0, size=(n, cols))).astype(np.float32)
            out[r:r + n] = f32_to_bf16_bits(t * colscale[None, :])
    elif cfg.kind == "weight":
        for r, n in _blocks(rows):
            out[r:r + n] = f32_to_bf16_bits(np.float32(0.02) * rng.standard_normal((n, cols), dtype=np.float32))
    elif cfg.kind == "gradient":
        for r, n in _blocks(rows):
            mag = (10.0 ** rng.uniform(-2.0, 2.0, size=(n, 1))).astype(np.float32)
            g = np.float32(1e-3) * rng.standard_normal((n, cols), dtype=np.float32)
            out[r:r + n] = f32_to_bf16_bits(g * mag)
    elif cfg.kind == "mixture":
        for r, n in _blocks(rows):
            sel = rng.random((n, cols), dtype=np.float32) < np.float32(0.7)
            nrm = rng.standard_normal((n, cols), dtype=np.float32)
            lap = rng.laplace(0.0, 1.0, size=(n, cols)).astype(np.float32)
            big = rng.random((n, cols), dtype=np.float32) < np.float32(0.001)
            v = np.where(sel, nrm, lap)
            v = np.where(big, v * np.float32(100.0), v)
            out[r:r + n] = f32_to_bf16_bits(v)
    else:  # pragma: no cover
        raise KeyError(cfg.kind)
    return out


def sha256(a: np.ndarray) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def edge_tensors() -> dict[str, np.ndarray]:
    """Small hand-built tensors for the degenerate cases (bf16 bit patterns)."""
    rng = np.random.Generator(np.random.PCG64(1234))
    cases: dict[str, np.ndarray] = {}
    cases["zeros_3x48"] = np.zeros((3, 48), dtype=np.uint16)
    one = np.zeros((4, 64), dtype=np.float32)
    one[2, 37] = -3.25
    cases["one_nonzero"] = f32_to_bf16_bits(one)
    cases["row1_col16"] = f32_to_bf16_bits(rng.standard_normal((1, 16), dtype=np.float32))
    last = rng.standard_normal((5, 80), dtype=np.float32)
    last[4, 79] = 1000.0
    cases["amax_last"] = f32_to_bf16_bits(last)
    tiny_row = rng.standard_normal((6, 96), dtype=np.float32)
    tiny_row[3] *= np.float32(2.0 ** -20)
    cases["tiny_row"] = f32_to_bf16_bits(tiny_row)
    pm0 = np.zeros((2, 32), dtype=np.uint16)
    pm0[0, ::2] = 0x8000
    pm0[1, 5] = 0x3F80
    pm0[1, 6] = 0x8000
    cases["signed_zeros"] = pm0
    # values on E2M1 rounding midpoints times a power-of-two scale (amax 6 -> d = 1)
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, -0.25, -0.75, -1.25, -1.75, -2.5, -3.5, -5.0, -6.0],
                    dtype=np.float32)
    cases["fp4_midpoints"] = f32_to_bf16_bits(np.tile(mids, (2, 3)))
    # integer-grid midpoints: k + 0.5 in units of 6/7 are not bf16 values; use halves of 7 -> d_int = 1
    ints = np.array([0.5, 1.5, 2.5, 3.5, 4.5, 5.5, 6.5, 7.0, -0.5, -1.5, -2.5, -3.5, -4.5, -5.5, -6.5, -7.0],
                    dtype=np.float32)
    cases["int4_midpoints"] = f32_to_bf16_bits(np.tile(ints, (2, 2)))
    huge = rng.standard_normal((4, 64), dtype=np.float32) * np.float32(1e37)
    huge[1, 1] = np.float32(3.38e38)
    cases["near_bf16_max"] = f32_to_bf16_bits(huge)
    small = rng.standard_normal((4, 64), dtype=np.float32) * np.float32(1e-25)
    cases["small_1e-25"] = f32_to_bf16_bits(small)
    wide = rng.standard_normal((8, 256), dtype=np.float32) * (10.0 ** rng.uniform(-6, 3, size=(8, 256))).astype(np.float32)
    cases["wide_dynamic_range"] = f32_to_bf16_bits(wide)
    ragged = rng.standard_normal((37, 16 * 13), dtype=np.float32)
    cases["ragged_37x208"] = f32_to_bf16_bits(ragged)
    # bf16 subnormal elements (bit patterns 0x0001..0x007F, both signs) under a normal tensor maximum: alone in
    # a group (zero scale), next to normal values, and as the only non-zero values of a row
    sub = f32_to_bf16_bits(rng.standard_normal((4, 64), dtype=np.float32))
    sub[0, :16] = rng.integers(1, 0x80, 16).astype(np.uint16) | (rng.integers(0, 2, 16).astype(np.uint16) << 15)
    sub[1, 16:24] = rng.integers(1, 0x80, 8).astype(np.uint16)
    sub[2, :] = 0
    sub[2, 5] = 0x0001
    sub[2, 40] = 0x807F
    cases["bf16_subnormals"] = sub
    # the smallest tensor maximum the library supports, 2^-100, and one a little above it
    for name, k in (("amax_2^-100", -100), ("amax_2^-96", -96)):
        t = rng.standard_normal((4, 64), dtype=np.float32)
        t = t / np.abs(t).max() * np.float32(2.0 ** k)
        cases[name] = f32_to_bf16_bits(t)
    return cases


def below_range_tensor() -> np.ndarray:
    """A tensor whose maximum, 2^-110, lies below the supported range (maximum 0 or at least 2^-100)."""
    rng = np.random.Generator(np.random.PCG64(4321))
    t = rng.standard_normal((4, 64), dtype=np.float32)
    return f32_to_bf16_bits(t / np.abs(t).max() * np.float32(2.0 ** -110))



def arbitrary_quantized_bytes(bits: int, group: int, rows: int = 16, cols: int = 1024, seed: int = 0):
    """Code and scale bytes that no quantizer produced, for the dequantize tests: random code bytes; every scale
    byte 0x00..0xFF occurs (rows 0 and 1 run through all of them); row 2 starts with the special bytes -- E4M3
    NaN with and without bit 7, 0x80, zero, the largest scale with and without bit 7, the smallest -- over code
    bytes that contain the most negative integer patterns and the FP code 'minus zero'."""
    rng = np.random.default_rng(100 + seed)
    codes = rng.integers(0, 256, (rows, cols * bits // 8), dtype=np.uint8)
    scales = rng.integers(0, 256, (rows, cols // group), dtype=np.uint8)
    scales[0, :] = np.arange(cols // group) % 256
    scales[1, :] = (255 - np.arange(cols // group)) % 256
    scales[2, :8] = [0x7F, 0xFF, 0x80, 0x00, 0x7E, 0xFE, 0x01, 0x81]
    codes[2, :16 * bits] = np.tile(np.frombuffer(bytes([0x88, 0x08, 0x80, 0x00, 0xFF, 0x77, 0x24, 0x92]), np.uint8), 2 * bits)
    return codes, scales

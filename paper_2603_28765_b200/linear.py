"""The quantized linear layer of the paper's training recipe (Sec. 4.1), emulated as the paper did it.

Weights, activations and gradients of a linear layer  Y = X W^T  (X [tokens, d_in], W [d_out, d_in]) are
quantized, dequantized to BF16 and multiplied with plain BF16 GEMMs.  Every operand is quantized along the
dimension its product contracts over:

    forward   Y  = q(X) q(W)^T            contraction over d_in:   rows of X, rows of W           round to nearest
    dgrad     dX = q(dY) q(W)             contraction over d_out:  rows of dY (stochastic rounding, 17/16 factor),
                                                                   columns of W                   round to nearest
    wgrad     dW = q(dY)^T q(X)           contraction over tokens: columns of dY (Hadamard, stochastic rounding,
                                                                   17/16 factor), columns of X (Hadamard)

The random Hadamard transform runs along the token dimension with one sign vector for both operands of the
weight-gradient product, so it cancels in the product (the 16-point block transform is orthogonal).  Stochastic
rounding is applied to activation gradients only; the 16/17 factor of Sec. 4.1 goes with it.

All format-specific work is one call of ``abs_quantize_dequantize`` per operand (the one-pass emulation, along
rows or down the columns, output in the operand's own orientation); the GEMMs are plain library calls.
"""
from __future__ import annotations

from . import binding as B


def emulate(x, fmt: int = B.ABS_FMT_IF4, *, columns: bool = False, hadamard: bool = False, stochastic: bool = False,
            sign_mask: int = 0, seed: int = 0):
    """bf16 tensor of the shape of ``x`` holding dequantize(quantize(x)); groups of 16 along the rows, or down
    the columns with ``columns``.  With ``hadamard`` the values are those of the transformed tensor."""
    flags = (B.ABS_F_GROUPS_DOWN_COLUMNS if columns else 0) | (B.ABS_F_HADAMARD16 if hadamard else 0)
    if stochastic:
        flags |= B.ABS_F_STOCHASTIC | B.ABS_F_SR_SCALE_17_16
    out, _ = B.abs_quantize_dequantize(fmt, x, opts=B.make_opts(flags, sign_mask, seed))
    return out


def _mm(a, b):
    """BF16 x BF16 -> BF16 product with FP32 accumulation."""
    import torch
    return torch.matmul(a, b)


def forward(x, w, fmt: int = B.ABS_FMT_IF4):
    """Y = q(X) q(W)^T; x [tokens, d_in], w [d_out, d_in], both bf16 CUDA tensors."""
    return _mm(emulate(x, fmt), emulate(w, fmt).t())


def backward(x, w, dy, fmt: int = B.ABS_FMT_IF4, *, sign_mask: int = 0x5A3C, seed: int = 0):
    """(dX, dW) for the layer above; dy [tokens, d_out] bf16.  Two different random streams are used for the
    two quantizations of dy (seed and seed + 1)."""
    dx = _mm(emulate(dy, fmt, stochastic=True, seed=seed), emulate(w, fmt, columns=True))
    dyq = emulate(dy, fmt, columns=True, hadamard=True, stochastic=True, sign_mask=sign_mask, seed=seed + 1)
    xq = emulate(x, fmt, columns=True, hadamard=True, sign_mask=sign_mask)
    dw = _mm(dyq.t(), xq)
    return dx, dw

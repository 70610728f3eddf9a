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

``forward_tc`` / ``backward_tc`` compute the same three products without the BF16 detour: every operand is quantized
once into codes and scales that are K-major for its product (``abs_quantize`` along the rows, ``abs_quantize_transposed``
down the columns) and the products run on the tensor cores with the MAC arithmetic of Sec. 5.2 (``abs_matmul``:
exact code products, FP32 scale path with the factors 6/7 and 36/49, FP32 accumulation and output).
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


# ----------------------------------------------------------------------------- the same layer on the tensor cores


def _opts(*, hadamard: bool = False, stochastic: bool = False, sign_mask: int = 0, seed: int = 0):
    flags = B.ABS_F_HADAMARD16 if hadamard else 0
    if stochastic:
        flags |= B.ABS_F_STOCHASTIC | B.ABS_F_SR_SCALE_17_16
    return B.make_opts(flags, sign_mask, seed) if flags else None


def forward_tc(x, w, fmt: int = B.ABS_FMT_IF4, *, bf16: bool = False, next_fmt: int | None = None):
    """Y = q(X) q(W)^T as float32 [tokens, d_out] (bfloat16 with ``bf16``, ready to be the next layer's input): both
    operands quantized along d_in, one ``abs_matmul``.  With ``next_fmt`` (implies bf16) the product kernel also leaves
    the tensor scale of Y for that format, and the call returns (Y, alpha): ``quantize_with(next_fmt, Y, alpha)`` then
    quantizes Y without a pass for its maximum.  d_out must be a multiple of 128, d_in of 256 (any number of tokens)."""
    tokens, d_in = x.shape
    d_out = w.shape[0]
    qx, qw = B.abs_quantize(fmt, x), B.abs_quantize(fmt, w)
    if next_fmt is not None:
        return B.abs_matmul(fmt, qx, qw, tokens, d_out, d_in, bf16=True, next_fmt=next_fmt)
    return B.abs_matmul(fmt, qx, qw, tokens, d_out, d_in, bf16=bf16)


def quantize_with(fmt: int, x, alpha):
    """abs_quantize of ``x`` with a tensor scale that is already known (a CUDA float32[1], e.g. from ``forward_tc`` with
    ``next_fmt``): the group-quantize kernel alone.  Returns (codes, scales, alpha)."""
    return B.abs_quantize(fmt, x, tensor_scale=alpha, opts=B.make_opts(B.ABS_F_ALPHA_GIVEN))


def backward_tc(x, w, dy, fmt: int = B.ABS_FMT_IF4, *, sign_mask: int = 0x5A3C, seed: int = 0):
    """(dX float32 [tokens, d_in], dW float32 [d_out, d_in]) with the recipe of ``backward``:
    dX = q(dY) q(W^T)^T contracts over d_out, dW = q(dY^T) q(X^T)^T over the tokens (Hadamard on both, stochastic
    rounding and the 17/16 factor on the gradient).  The transposed operands come from ``abs_quantize_transposed``,
    which writes them K-major without materialising a transpose.  All three sizes multiples of 256."""
    tokens, d_in = x.shape
    d_out = w.shape[0]
    q_dy = B.abs_quantize(fmt, dy, opts=_opts(stochastic=True, seed=seed))                 # [tokens, d_out] along d_out
    q_wt = B.abs_quantize_transposed(fmt, w)                                                # W^T [d_in, d_out] along d_out
    dx = B.abs_matmul(fmt, q_dy, q_wt, tokens, d_in, d_out)
    q_dyt = B.abs_quantize_transposed(fmt, dy, opts=_opts(hadamard=True, stochastic=True, sign_mask=sign_mask,
                                                          seed=seed + 1))                  # dY^T [d_out, tokens]
    q_xt = B.abs_quantize_transposed(fmt, x, opts=_opts(hadamard=True, sign_mask=sign_mask))  # X^T [d_in, tokens]
    dw = B.abs_matmul(fmt, q_dyt, q_xt, d_out, d_in, tokens)
    return dx, dw

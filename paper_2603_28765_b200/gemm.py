"""Matrix products of IF4-quantized operands, two ways (paper Sec. 4.1 and Sec. 5.2).

Both take operands quantized along K: A as [M, K], B as [N, K] (codes, scales, alpha from
``abs_quantize``) and return C = A B^T as a CUDA float32 [M, N] tensor.

``matmul_emulated``  what the paper's experiments ran (Sec. 4.1): dequantize to FP32, round to BF16,
                     one BF16 GEMM with FP32 accumulation.
``matmul_mac``       the arithmetic of the paper's IF4 MAC unit (Sec. 5.2): inside a pair of groups the
                     decoded 4-bit values are multiplied and summed, and the pair's scale product gets the
                     factor 1, 6/7 or 36/49 (none, one, both groups stored as integers) in FP32 on the
                     scale path.  This is the library's own tensor-core kernel (``abs_matmul``: block-scaled
                     FP4 MMAs on the codes themselves, three accumulators, factors in the FP32 epilogue)
                     whenever N is a multiple of 128 and K of 256 (any M).
``matmul_mac_split`` the same arithmetic for any shape, and the cross-check of the kernel above, from parts
                     that are exact in BF16: the library's split dequantize produces, for each operand, the
                     FP-group part and the raw integer-group part -- each a 4-bit code times an E4M3 scale,
                     hence EXACT in BF16 -- and four plain BF16 tensor-core GEMMs (FP32 accumulation, every
                     product exact) are combined with the FP32 factors:
                         C = A_F B_F^T + 6/7 (A_F B_I^T + A_I B_F^T) + 36/49 A_I B_I^T,  times alpha_a alpha_b.

In ``matmul_emulated`` and ``matmul_mac_split`` the GEMMs are plain library calls (torch.mm -> cuBLAS);
``matmul_mac`` contracts in this library's own kernel.
"""
from __future__ import annotations

from . import binding as B

FMT = B.ABS_FMT_IF4


def _deq(q, rows, k, flags=0, unit_alpha=False):
    import torch
    codes, scales, alpha = q
    if unit_alpha:
        alpha = torch.ones(1, dtype=torch.float32, device=codes.device)
    return B.abs_dequantize(FMT, codes, scales, alpha, rows, k, opts=B.make_opts(flags) if flags else None)


def matmul_emulated(qa, qb, m: int, n: int, k: int):
    """Sec. 4.1 emulation: BF16(dequantize(A)) @ BF16(dequantize(B))^T with FP32 accumulation."""
    import torch
    a = _deq(qa, m, k)
    b = _deq(qb, n, k)
    return _mm_fp32(a, b)


def matmul_mac(qa, qb, m: int, n: int, k: int):
    """Sec. 5.2 MAC arithmetic: the library's tcgen05 kernel where the shape allows, else the BF16 split."""
    if n % 128 == 0 and k % 256 == 0:
        return B.abs_matmul(FMT, qa, qb, m, n, k)
    return matmul_mac_split(qa, qb, m, n, k)


def matmul_mac_split(qa, qb, m: int, n: int, k: int):
    """Sec. 5.2 MAC arithmetic via the exact BF16 split (see the module docstring)."""
    import torch
    a_f = _deq(qa, m, k, B.ABS_F_FP_GROUPS_ONLY, unit_alpha=True)
    a_i = _deq(qa, m, k, B.ABS_F_INT_GROUPS_RAW, unit_alpha=True)
    b_f = _deq(qb, n, k, B.ABS_F_FP_GROUPS_ONLY, unit_alpha=True)
    b_i = _deq(qb, n, k, B.ABS_F_INT_GROUPS_RAW, unit_alpha=True)
    mm = _mm_fp32
    c67 = torch.tensor(6.0, dtype=torch.float32) / torch.tensor(7.0, dtype=torch.float32)
    c3649 = torch.tensor(36.0, dtype=torch.float32) / torch.tensor(49.0, dtype=torch.float32)
    c = mm(a_f, b_f) + c67.item() * (mm(a_f, b_i) + mm(a_i, b_f)) + c3649.item() * mm(a_i, b_i)
    return c * (qa[2].float() * qb[2].float())


def _mm_fp32(x, y):
    """BF16 x BF16 -> FP32 output with FP32 accumulation (the products of the split halves are exact)."""
    import torch
    try:
        return torch.mm(x, y.t(), out_dtype=torch.float32)
    except TypeError:                     # older torch: accumulate in FP32 by promoting the operands
        return torch.mm(x.float(), y.float().t())

"""Quantization bias under stochastic rounding (paper App. B), measured on the GPU path.

A gradient-like tensor is quantized with stochastic rounding under many seeds; the mean of the
dequantized values minus the input, as a function of the input's magnitude, shows whether the format
is biased.  The paper's observation: NVFP4 with stochastic rounding is unbiased, while IF4 -- which
selects between two stochastically rounded candidates -- pushes the largest values slightly up, and
only very few values are affected.

    python -m paper_2603_28765_b200.sr_bias [--trials 1000] [--rows 2048] [--no-scale-option]

The tensor is the synthetic gradient configuration (N(0,1e-6) times per-row 10^U(-2,2)); the paper used
gradients of its own training runs, which need its models.  Prints one JSON line per format with, per
magnitude bin (|x| relative to the largest |x| of its group of 16), the mean signed change in units of
the group maximum and the share of elements in the bin.
"""
from __future__ import annotations

import argparse
import json

import numpy as np


def run(trials: int, rows: int, cols: int, scale_option: bool, device: str = "cuda"):
    import torch
    from . import binding as B
    from . import inputs as I

    xb = I.generate("cfg4", rows, cols)
    x = torch.from_numpy(xb.view(np.int16)).to(device).view(torch.bfloat16)
    xf = x.float()
    flags = B.ABS_F_STOCHASTIC | (B.ABS_F_SR_SCALE_17_16 if scale_option else 0)
    fp32 = B.make_opts(B.ABS_F_OUT_FP32)
    gmax = xf.abs().view(rows, cols // 16, 16).amax(dim=2, keepdim=True).clamp_min(1e-30)
    rel = (xf.abs().view(rows, cols // 16, 16) / gmax).reshape(rows, cols)
    sign = torch.sign(xf)
    edges = torch.tensor([0.0, 0.1, 0.2, 0.3, 0.4, 0.5, 0.6, 0.7, 0.8, 0.9, 1.0 + 1e-6], device=device)
    out = {}
    for name, fmt in (("nvfp4", B.ABS_FMT_NVFP4), ("if4", B.ABS_FMT_IF4)):
        acc = torch.zeros_like(xf, dtype=torch.float64)
        codes = scales = ts = None
        deq = torch.empty_like(xf)
        for seed in range(trials):
            codes, scales, ts = B.abs_quantize(fmt, x, codes, scales, ts, opts=B.make_opts(flags, 0, seed))
            B.abs_dequantize(fmt, codes, scales, ts, rows, cols, out=deq, opts=fp32)
            acc += deq
        # outward (magnitude-increasing) change of the mean, in units of the group maximum
        bias = ((acc / trials - xf.double()) * sign).view(rows, cols // 16, 16) / gmax
        bias = bias.reshape(rows, cols)
        bins = []
        for lo, hi in zip(edges[:-1], edges[1:]):
            m = (rel >= lo) & (rel < hi)
            cnt = int(m.sum())
            bins.append({"rel_lo": round(float(lo), 2), "rel_hi": round(min(float(hi), 1.0), 2),
                         "share": cnt / rel.numel(), "mean_change_over_gmax": float(bias[m].mean()) if cnt else 0.0})
        out[name] = bins
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--trials", type=int, default=1000)
    ap.add_argument("--rows", type=int, default=2048)
    ap.add_argument("--cols", type=int, default=8192)
    ap.add_argument("--no-scale-option", action="store_true", help="without the 17/16 scale option of Sec. 4.1")
    a = ap.parse_args()
    res = run(a.trials, a.rows, a.cols, not a.no_scale_option)
    for name, bins in res.items():
        print(json.dumps({"format": name, "trials": a.trials, "scale_option_17_16": not a.no_scale_option, "bins": bins}))


if __name__ == "__main__":
    main()

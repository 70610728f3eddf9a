"""Per-configuration throughput table of the library's kernels (run on a B200 machine).

    python -m paper_2603_28765_b200.report [--quick] [--only CFG[:FMT]] [--rows R] [--transposed] [--matmul]

``--only cfg4:if4 --rows 4096 --quick`` restricts the run to one configuration (and format) at a reduced
row count: the small case to put under a profiler.

For every benchmark configuration and format it times, with CUDA events over back-to-back calls
that rotate over enough buffer sets to defeat L2 reuse between calls:
  T1  the group-quantize kernel alone (alpha given)          bytes = 2N + codes + scales
  T2  abs_quantize end to end (amax pass + group-quantize)   bytes = 4N + codes + scales (DRAM basis)
  T3  abs_dequantize                                         bytes = codes + scales + 2N
  T4  abs_quantize_dequantize (amax pass + one-pass emulation, no code outputs)
and prints one JSON line per row, with the same three figures for a warm L2 (one buffer set reused) and the
first 16 hex digits of the SHA-256 of the first input set and of its codes and scale bytes.  With ``--transposed`` it times abs_quantize_transposed instead (the kernel
alone, alpha given; the same bytes move), for IF4 and NVFP4 with and without the gradient options.  Inputs are random bf16 tensors of the configuration's shape
(timing does not depend on the values beyond the INT/FP mix); parity is the test suite's job.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json


def main():
    import torch
    from . import binding as B

    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true", help="fewer repetitions")
    ap.add_argument("--only", default="", help="one configuration, optionally one format: cfg4 or cfg4:if4")
    ap.add_argument("--rows", type=int, default=0, help="override the row count (smaller case for profiling)")
    ap.add_argument("--transposed", action="store_true", help="time abs_quantize_transposed (groups down the columns)")
    ap.add_argument("--linear", action="store_true", help="time the quantized linear layer (forward + backward), tensor-core and emulated routes")
    ap.add_argument("--matmul", action="store_true", help="time abs_matmul (square sizes; --rows picks one size)")
    args = ap.parse_args()
    L = B.lib()
    reps = 10 if args.quick else 40

    def loop_time(fn, n=reps, warm=3):
        for i in range(warm):
            fn(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(n):
            fn(i)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    def digest(t):
        import hashlib
        return hashlib.sha256(t.cpu().numpy().tobytes()).hexdigest()[:16]

    H, S, S17 = B.ABS_F_HADAMARD16, B.ABS_F_STOCHASTIC, B.ABS_F_SR_SCALE_17_16
    rows_cfg = [
        ("cfg2", 8192, 4096, [("if4", 0)]),
        ("cfg3a", 4096, 14336, [("if4", 0), ("nvfp4", 0)]),
        ("cfg3b", 14336, 4096, [("if4", 0), ("nvfp4", 0)]),
        ("cfg4", 16384, 8192, [("if4", H | S | S17), ("if4", H | S), ("if4", S), ("if4", H), ("nvfp4", H | S | S17)]),
        ("cfg5", 16384, 8192, [("if3", 0), ("if4", 0), ("if6_e2m3", 0), ("if6_e3m2", 0), ("nvfp4", 0),
                               ("if4_bs8", 0), ("if3_bs8", 0), ("nvfp4_bs8", 0)]),
    ]
    sp = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    only_cfg, _, only_fmt = args.only.partition(":")
    if args.matmul:
        # abs_matmul (tcgen05 kernel, Sec. 5.2 arithmetic) against the split path built from cuBLAS GEMMs and the
        # BF16 emulation of Sec. 4.1; operands N(0,1) and N(0, 0.02^2)
        from . import gemm
        for size in ([args.rows] if args.rows else [2048, 4096, 8192]):
            m = n = kk = size
            x = torch.randn(m, kk, device="cuda").to(torch.bfloat16)
            w = (torch.randn(n, kk, device="cuda") * 0.02).to(torch.bfloat16)
            for fname in ("if4", "nvfp4"):
                fmt = B.FMT_NAMES[fname]
                qa, qb = B.abs_quantize(fmt, x), B.abs_quantize(fmt, w)
                ws = torch.empty(L.abs_matmul_workspace_bytes(fmt, m, n, kk) + 1024, dtype=torch.uint8, device="cuda")
                out = torch.empty((m, n), dtype=torch.float32, device="cuda")
                t = loop_time(lambda i: B.abs_matmul(fmt, qa, qb, m, n, kk, out=out, workspace=ws))
                B.abs_matmul(fmt, qa, qb, m, n, kk, out=out, workspace=ws, check=True)
                row = {"matmul": [m, n, kk], "fmt": fname, "abs_matmul_ms": round(t, 4),
                       "useful_TFLOPs": round(2.0 * m * n * kk / t / 1e9, 1),
                       "mma_TFLOPs": round((9 if fname == "if4" else 1) * 2.0 * m * n * kk / t / 1e9, 1)}
                if fname == "if4":
                    row["split_path_cublas_ms"] = round(loop_time(lambda i: gemm.matmul_mac_split(qa, qb, m, n, kk)), 4)
                    row["bf16_emulation_ms"] = round(loop_time(lambda i: gemm.matmul_emulated(qa, qb, m, n, kk)), 4)
                    ref = gemm.matmul_mac_split(qa, qb, m, n, kk)
                    row["max_diff_vs_split_path"] = float((out - ref).abs().max() / ref.abs().max())
                print(json.dumps(row), flush=True)
        return
    if args.linear:
        # the quantized linear layer of Sec. 4.1 (forward, dgrad, wgrad with the gradient options): tensor-core route
        # (quantize to K-major codes + abs_matmul) against the emulated route (one-pass emulation + cuBLAS BF16 GEMMs)
        from . import linear
        tokens, d_in, d_out = (args.rows or 8192), 4096, 14336
        x = torch.randn(tokens, d_in, device="cuda").to(torch.bfloat16)
        w = (torch.randn(d_out, d_in, device="cuda") * 0.02).to(torch.bfloat16)
        dy = (torch.randn(tokens, d_out, device="cuda") * 1e-3).to(torch.bfloat16)
        for fname in ("if4", "nvfp4"):
            fmt = B.FMT_NAMES[fname]
            row = {"linear": {"tokens": tokens, "d_in": d_in, "d_out": d_out}, "fmt": fname,
                   "forward_tc_ms": round(loop_time(lambda i: linear.forward_tc(x, w, fmt)), 4),
                   "backward_tc_ms": round(loop_time(lambda i: linear.backward_tc(x, w, dy, fmt)), 4),
                   "forward_emulated_ms": round(loop_time(lambda i: linear.forward(x, w, fmt)), 4),
                   "backward_emulated_ms": round(loop_time(lambda i: linear.backward(x, w, dy, fmt)), 4),
                   "bf16_gemms_alone_ms": round(loop_time(lambda i: (torch.matmul(x, w.t()), torch.matmul(dy, w),
                                                                     torch.matmul(dy.t(), x))), 4),
                   "gemm_flops": 6.0 * tokens * d_in * d_out}
            y, ye = linear.forward_tc(x, w, fmt), linear.forward(x, w, fmt).float()
            row["forward_tc_vs_emulated_rel"] = float((y - ye).norm() / y.norm())
            print(json.dumps(row), flush=True)
        return
    if args.transposed:
        for name, rows, cols in (("cfg2", 8192, 4096), ("cfg4", 16384, 8192)):
            if only_cfg and name != only_cfg:
                continue
            if args.rows:
                rows = args.rows
            n = rows * cols
            k = max(4, int(1.0e9 // (n * 2)))
            xs = [torch.randn(rows, cols, device="cuda").to(torch.bfloat16) for _ in range(k)]
            codes = [torch.empty(n // 2, dtype=torch.uint8, device="cuda") for _ in range(k)]
            scales = [torch.empty(n // 16, dtype=torch.uint8, device="cuda") for _ in range(k)]
            ts = [torch.full((1,), 0.01, dtype=torch.float32, device="cuda") for _ in range(k)]
            for fname, flags in (("if4", 0), ("nvfp4", 0), ("if4", H), ("if4", H | S | S17), ("nvfp4", H | S | S17)):
                if only_fmt and fname != only_fmt:
                    continue
                fmt = B.FMT_NAMES[fname]
                og = B.make_opts(flags | B.ABS_F_ALPHA_GIVEN, 0x5A3C, 1234)
                a = [(fmt, xs[i].data_ptr(), rows, cols, codes[i].data_ptr(), scales[i].data_ptr(), ts[i].data_ptr(),
                      C.byref(og), sp) for i in range(k)]
                t = loop_time(lambda i: L.abs_quantize_transposed(*a[i % k]))
                opt = "+".join(s for s, f in (("hadamard", H), ("sr", S), ("17/16", S17)) if flags & f) or "rtn"
                print(json.dumps({"config": name, "shape": [rows, cols], "fmt": fname, "options": opt, "transposed": True,
                                  "T1_quantize_kernel_us": round(t * 1e3, 1),
                                  "T1_GBs": round(2.5625 * n / t / 1e6)}), flush=True)
            del xs, codes, scales
        return
    for name, rows, cols, variants in rows_cfg:
        if only_cfg and name != only_cfg:
            continue
        if only_fmt:
            variants = [v for v in variants if v[0] == only_fmt]
        if args.rows:
            rows = args.rows
        n = rows * cols
        k = max(4, int(1.0e9 // (n * 2)))
        xs = [(torch.randn(rows, cols, device="cuda") * (1 + 3 * torch.rand(rows, 1, device="cuda"))).to(torch.bfloat16)
              for _ in range(k)]
        for fname, flags in variants:
            fmt = B.FMT_NAMES[fname]
            bits = B.FMT_BITS[fmt]
            codes = [torch.empty(n * bits // 8, dtype=torch.uint8, device="cuda") for _ in range(k)]
            scales = [torch.empty(n // B.FMT_GROUP[fmt], dtype=torch.uint8, device="cuda") for _ in range(k)]
            ts = [torch.zeros(1, dtype=torch.float32, device="cuda") for _ in range(k)]
            outs = [torch.empty(rows, cols, dtype=torch.bfloat16, device="cuda") for _ in range(min(k, 4))]
            o_full = B.make_opts(flags, 0x5A3C, 1234)
            o_given = B.make_opts(flags | B.ABS_F_ALPHA_GIVEN, 0x5A3C, 1234)
            for i in range(k):
                B.abs_quantize(fmt, xs[i], codes[i], scales[i], ts[i], opts=o_full)
            torch.cuda.synchronize()
            qa = [(fmt, xs[i].data_ptr(), rows, cols, codes[i].data_ptr(), scales[i].data_ptr(), ts[i].data_ptr(),
                   C.byref(o_given), sp) for i in range(k)]
            fa = [(fmt, xs[i].data_ptr(), rows, cols, codes[i].data_ptr(), scales[i].data_ptr(), ts[i].data_ptr(),
                   C.byref(o_full), sp) for i in range(k)]
            da = [(fmt, codes[i].data_ptr(), scales[i].data_ptr(), ts[i].data_ptr(), rows, cols,
                   outs[i % len(outs)].data_ptr(), sp) for i in range(k)]
            t1 = loop_time(lambda i: L.abs_quantize_ex(*qa[i % k]))
            t2 = loop_time(lambda i: L.abs_quantize_ex(*fa[i % k]))
            t3 = loop_time(lambda i: L.abs_dequantize(*da[i % k]))
            # warm L2: the same buffer set every call (tensors up to about 100 MB stay in the 126 MB L2)
            t1w = loop_time(lambda i: L.abs_quantize_ex(*qa[0]))
            t2w = loop_time(lambda i: L.abs_quantize_ex(*fa[0]))
            t3w = loop_time(lambda i: L.abs_dequantize(*da[0]))
            # fingerprints of what was timed: SHA-256 of the first input set and of its outputs
            L.abs_quantize_ex(*fa[0])
            torch.cuda.synchronize()
            sha = {"input": digest(xs[0].view(torch.int16)), "codes": digest(codes[0]), "scales": digest(scales[0])}
            t4 = None
            if fmt in (B.ABS_FMT_NVFP4, B.ABS_FMT_IF4) or not (flags & (H | S)):
                ea = [(fmt, xs[i].data_ptr(), rows, cols, outs[i % len(outs)].data_ptr(), None, None, ts[i].data_ptr(),
                       C.byref(o_full), sp) for i in range(k)]
                t4 = loop_time(lambda i: L.abs_quantize_dequantize(*ea[i % k]))
            outb = n * bits / 8 + n / B.FMT_GROUP[fmt]
            opt = "+".join(s for s, f in (("hadamard", H), ("sr", S), ("17/16", S17)) if flags & f) or "rtn"
            print(json.dumps({
                "config": name, "shape": [rows, cols], "fmt": fname, "options": opt,
                "T1_quantize_kernel_us": round(t1 * 1e3, 1), "T1_GBs": round((2 * n + outb) / t1 / 1e6),
                "T1_pct_of_8000": round((2 * n + outb) / t1 / 1e6 / 80.0, 1),
                "T2_dram_basis_pct_of_8000": round((4 * n + outb) / t2 / 1e6 / 80.0, 1),
                "T2_abs_quantize_us": round(t2 * 1e3, 1), "T2_dram_basis_GBs": round((4 * n + outb) / t2 / 1e6),
                "T2_effective_GBs": round((2 * n + outb) / t2 / 1e6),
                "T3_dequantize_us": round(t3 * 1e3, 1), "T3_GBs": round((2 * n + outb) / t3 / 1e6),
                "T4_quantize_dequantize_us": round(t4 * 1e3, 1) if t4 else None,
                "elements_per_s_T2": round(n / (t2 * 1e-3)),
                "warm_l2_us": {"T1": round(t1w * 1e3, 1), "T2": round(t2w * 1e3, 1), "T3": round(t3w * 1e3, 1)},
                "sha256_16": sha,
            }), flush=True)
            del codes, scales, outs
        del xs


if __name__ == "__main__":
    main()

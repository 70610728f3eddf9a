#!/usr/bin/env python
"""Benchmark of the IF4 quantize + dequantize hot path on B200.

A step is one pass of the whole path over one tensor of the LLM-activation-like workload
(bf16 8192 x 4096, 0.5*Student-t(3) with 0.5 % outlier columns x50): ``abs_quantize`` (grid-wide
amax -> alpha, then the group-quantize kernel) followed by ``abs_dequantize`` -- three kernel
launches.  The metric is GB/s of algorithmic bytes in + out per step:
    quantize   2N (bf16 in) + N/2 (codes) + N/16 (scales)
    dequantize N/2 + N/16 in, 2N (bf16 out)                    => 5.125 N bytes per step.
Steps rotate over enough tensor sets that the inputs alone exceed 4x the L2 capacity, so every step starts cold.
Before the timed region an untimed loop of the same steps runs for about 250 ms so that the clocks are up
(disclosed as `clock_ramp_ms`); the timed region is exactly K steps.  The dominant kernel is timed separately in
5 batches of 100 launches whatever K is (median, best and worst reported).

  python bench.py [--gpus N] [--steps K] [--warmup W]          CUDA path, one JSON line
  python bench.py --impl reference ...                         the CPU oracle timed on host cores

With N > 1 (launched by torch.distributed.run) every rank runs the same step on its own tensors:
independent problems, no data-path collective, weak scaling; time = max over ranks.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2603_28765_b200 import inputs as I  # noqa: E402

WORKLOAD = "cfg2"
FMT_IF4 = 1
METRIC = "IF4 quantize+dequantize GB/s (algorithmic bytes in+out)"
UNIT = "GB/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0

TRAFFIC_FILE = os.path.join(ROOT, "profiles", "quantize4_fast_if4_cfg2_traffic.txt")
CLOCK_RAMP_MS = 250.0           # untimed steps run right before the timed region so that it starts at full clocks
KERNEL_BATCHES = 5              # the dominant kernel is timed in this many batches ...
KERNEL_BATCH_LAUNCHES = 100     # ... of this many back-to-back launches each, whatever --steps is


def ncu_traffic(n_elems: int):
    """DRAM bytes per launch of the group-quantize kernel from the tracked ncu summary (dram__bytes_read.sum +
    dram__bytes_write.sum of one capture, scaled by the element count), and the commit it was captured at."""
    try:
        kv = {}
        with open(TRAFFIC_FILE) as f:
            for line in f:
                if ":" in line and not line.lstrip().startswith("#"):
                    k, v = line.split(":", 1)
                    kv[k.strip()] = v.strip()
        per_elem = (float(kv["dram_bytes_read"]) + float(kv["dram_bytes_write"])) / float(kv["elements"])
        return per_elem * n_elems, kv.get("commit", "unknown")
    except Exception:
        return None, None


def step_bytes(n_elems: int) -> float:
    return 2.0 * (2.0 * n_elems + n_elems / 2.0 + n_elems / 16.0)


def quant_kernel_bytes(n_elems: int) -> float:
    return 2.0 * n_elems + n_elems / 2.0 + n_elems / 16.0


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def bf16_tensor_peak():
    """(TFLOP/s, source): the measured cuBLAS bf16 burst rate, else the recipe's fallback."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["bf16_tflops"]), "measured (MEASURED_PEAKS.json bf16_tflops, burst)"
    except Exception:
        return 1590.0, "fallback (1.59 PFLOP/s, earlier measurement on this pool)"


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML, each sample with its host timestamp,
    from before the clock-ramp loop until after the timed region; the report keeps the samples whose
    timestamps fall inside the timed window."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, torch_device_index: int, period_s: float = 0.0004):
        self.samples, self.max_mhz, self.ok = [], None, False      # samples: (t, sm_mhz, reason bits)
        self.period_s = period_s
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except TypeError:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # NVML missing: report that rather than guess
            self.err = repr(e)

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                self.samples.append((time.perf_counter(), mhz, r))
            except Exception:
                pass
            time.sleep(self.period_s)

    def start(self):
        if self.ok:
            self._stop.clear()
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
            self._thread = None

    def summary(self, t0: float, t1: float):
        """Clocks seen between host times t0 and t1 (the timed window)."""
        if not self.ok:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable: " + getattr(self, "err", "")}
        inside = [(m, r) for (t, m, r) in self.samples if t0 <= t <= t1]
        note = "samples inside the timed window"
        if not inside and self.samples:
            # the window was shorter than one NVML query: keep the two samples that bracket it
            before = [x for x in self.samples if x[0] < t0][-1:]
            after = [x for x in self.samples if x[0] > t1][:1]
            inside = [(m, r) for (_, m, r) in before + after]
            note = "timed window shorter than one NVML query: the samples taken just before and just after it"
        reasons = set()
        for _, r in inside:
            for bit, name in self.REASONS.items():
                if r & bit:
                    reasons.add(name)
        mhz = [m for m, _ in inside]
        return {"sm_mhz": int(statistics.median(mhz)) if mhz else None, "sm_min_mhz": min(mhz) if mhz else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(reasons), "samples": len(inside),
                "window_ms": round((t1 - t0) * 1e3, 3), "note": note}


# ----------------------------------------------------------------------------- CPU oracle legs

def oracle_rate(xb: np.ndarray, repeats: int, threads: int):
    """Times the oracle (quantize + dequantize, as it stands) on host cores; returns best GB/s and seconds."""
    from oracle import abs_oracle as O
    rows, cols = xb.shape
    best = float("inf")
    for _ in range(repeats):
        t0 = time.perf_counter()
        c, s, a = O.quantize(FMT_IF4, xb, threads=threads)
        O.dequantize(FMT_IF4, c, s, a, rows, cols, threads=threads)
        best = min(best, time.perf_counter() - t0)
    return step_bytes(rows * cols) / best / 1e9, best


def run_reference(args):
    """The reference arm: the CPU oracle on the same workload, metric and unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = I.CONFIGS[WORKLOAD]
    threads = os.cpu_count() or 1
    total = args.steps + args.warmup
    probe = I.generate(WORKLOAD, 256, cfg.cols)
    _, t_probe = oracle_rate(probe, 1, threads)
    budget_s = 120.0
    rows = int(min(cfg.rows, max(256, (budget_s / max(total, 1)) / (t_probe / 256))))
    rows -= rows % 64
    xb = I.generate(WORKLOAD, rows, cfg.cols)
    from oracle import abs_oracle as O
    times = []
    for i in range(total):
        t0 = time.perf_counter()
        c, s, a = O.quantize(FMT_IF4, xb, threads=threads)
        O.dequantize(FMT_IF4, c, s, a, rows, cfg.cols, threads=threads)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
    mean_s = sum(times) / len(times)
    value = step_bytes(rows * cfg.cols) / mean_s / 1e9
    sample = f"first {rows} of {cfg.rows} rows of the {cfg.rows}x{cfg.cols} tensor per step, {threads} threads over rows"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(mean_s * 1e3, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{WORKLOAD}: IF4 quantize+dequantize, bf16 {cfg.rows}x{cfg.cols}, {cfg.note}",
                   "sample": sample},
        "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }), flush=True)


# ----------------------------------------------------------------------------- CUDA path

def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2603_28765_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    L = B.lib()                       # raises if the CUDA library is missing
    B.abs_init(local)

    cfg = I.CONFIGS[WORKLOAD]
    rows, cols = cfg.rows, cfg.cols
    n = rows * cols
    nb_codes, nb_scales = B.abs_codes_bytes(FMT_IF4, rows, cols), B.abs_scales_bytes(FMT_IF4, rows, cols)
    set_bytes = 2 * n + nb_codes + nb_scales + 2 * n
    n_sets = max(2, -(-4 * L2_BYTES // (2 * n)))            # the INPUTS alone rotate over >= 4x L2 (8 sets here)

    # Synthetic inputs: one host tensor per rank from the seeded recipe; the other sets are row
    # rotations of it (same distribution, different addresses and group contents).
    xb = I.generate(WORKLOAD, seed=cfg.seed + 1000 * rank)
    x0 = torch.from_numpy(xb.view(np.int16)).to(dev).view(torch.bfloat16)
    xs = [x0] + [torch.roll(x0, shifts=17 * k, dims=0).contiguous() for k in range(1, n_sets)]
    codes = [torch.empty(nb_codes, dtype=torch.uint8, device=dev) for _ in range(n_sets)]
    scales = [torch.empty(nb_scales, dtype=torch.uint8, device=dev) for _ in range(n_sets)]
    alphas = [torch.zeros(1, dtype=torch.float32, device=dev) for _ in range(n_sets)]
    outs = [torch.empty((rows, cols), dtype=torch.bfloat16, device=dev) for _ in range(n_sets)]
    stream = torch.cuda.current_stream()
    sp = C.c_void_p(stream.cuda_stream)
    qargs = [(FMT_IF4, xs[k].data_ptr(), rows, cols, codes[k].data_ptr(), scales[k].data_ptr(), alphas[k].data_ptr(), sp)
             for k in range(n_sets)]
    dargs = [(FMT_IF4, codes[k].data_ptr(), scales[k].data_ptr(), alphas[k].data_ptr(), rows, cols, outs[k].data_ptr(), sp)
             for k in range(n_sets)]

    def step(i):
        k = i % n_sets
        rc = L.abs_quantize(*qargs[k])
        rc |= L.abs_dequantize(*dargs[k])
        if rc:
            raise RuntimeError(f"C-ABI call failed with status {rc}")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def event_pair():
        return torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_batches(fn, batches, launches, warm=8):
        """Average time per call (ms) of `batches` back-to-back loops of `launches` calls each, every loop between
        two CUDA events on the launching stream.  Returns the list of per-batch averages."""
        for i in range(warm):
            fn(i)
        torch.cuda.synchronize()
        res = []
        for b in range(batches):
            e0, e1 = event_pair()
            e0.record(stream)
            for i in range(launches):
                fn(b * launches + i)
            e1.record(stream)
            torch.cuda.synchronize()
            res.append(e0.elapsed_time(e1) / launches)
        return res

    sampler = ClockSampler(local)
    sampler.start()

    # ---- W warm-up steps, then an untimed clock-ramp loop of the same steps: a GPU that idled before the run
    # needs a few hundred milliseconds of load to reach its full clocks, and the timed region must not pay for it.
    warm = max(args.warmup, 3)
    for i in range(warm):
        step(i)
    barrier()
    ramp_t0 = time.perf_counter()
    ramp_steps = 0
    while not args.no_ramp and (time.perf_counter() - ramp_t0) * 1e3 < CLOCK_RAMP_MS:
        for i in range(64):
            step(ramp_steps + i)
        ramp_steps += 64
        torch.cuda.synchronize()
    clock_ramp_ms = (time.perf_counter() - ramp_t0) * 1e3
    barrier()

    # ---- timed region: exactly K steps between two events on the launching stream
    start, end = event_pair()
    t_host0 = time.perf_counter()
    start.record(stream)
    for i in range(args.steps):
        step(i)
    end.record(stream)
    barrier()
    t_host1 = time.perf_counter()
    ms_total = start.elapsed_time(end)
    clocks = sampler.summary(t_host0, t_host1)
    t = torch.tensor([ms_total], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_total = float(t.item())
    ms_per_step = ms_total / args.steps
    value = world * step_bytes(n) / (ms_per_step * 1e-3) / 1e9

    # ---- the same steps once more in batches, for the median next to the figure above (not part of `value`)
    step_batches = timed_batches(step, KERNEL_BATCHES, KERNEL_BATCH_LAUNCHES, warm=0)

    # ---- the in-step view of the group-quantize kernel: events recorded by the library right before and after it
    # on a few steps.  An event between two kernels of a step breaks their programmatic launch overlap, so the
    # interval contains the kernel's launch latency; it is reported beside the figure used for the roofline.
    probes = [event_pair() for _ in range(16)]
    for a, b in probes:        # torch creates the CUDA event on first record; the library re-records it later
        a.record(stream)
        b.record(stream)
    torch.cuda.synchronize()
    for pi, pr in enumerate(probes):
        for i in range(7):
            step(8 * pi + i)
        B.abs_profile_events(*pr)
        step(8 * pi + 7)
        B.abs_profile_events()
    torch.cuda.synchronize()
    in_step_ms = statistics.median(a.elapsed_time(b) for a, b in probes)

    # ---- the dominant kernel on its own: back-to-back launches of the group-quantize kernel over the same
    # rotating buffer sets (alpha given = the alpha the steps just produced, so only that kernel runs), in
    # KERNEL_BATCHES loops of KERNEL_BATCH_LAUNCHES launches whatever --steps is.  The median batch is the
    # figure used for the roofline; best and worst are printed beside it.
    og = B.make_opts(B.ABS_F_ALPHA_GIVEN)
    gargs = [(FMT_IF4, xs[k].data_ptr(), rows, cols, codes[k].data_ptr(), scales[k].data_ptr(), alphas[k].data_ptr(),
              C.byref(og), sp) for k in range(n_sets)]
    q_batches = timed_batches(lambda i: L.abs_quantize_ex(*gargs[i % n_sets]), KERNEL_BATCHES, KERNEL_BATCH_LAUNCHES)
    q_ms = statistics.median(q_batches)
    peak, peak_src = measured_peak()
    achieved = quant_kernel_bytes(n) / (q_ms * 1e-3) / 1e9
    traffic, traffic_commit = ncu_traffic(n)
    roofline = {"bound": "hbm", "kernel": "quantize4_fast_kernel<IF4> (group-quantize, Fig. 3a steps 1-10)",
                "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4),
                "peak_source": peak_src, "frac_of_nominal_8000_gbs": round(achieved / 8000.0, 4),
                "us_per_launch": round(q_ms * 1e3, 2), "us_per_launch_best": round(min(q_batches) * 1e3, 2),
                "us_per_launch_worst": round(max(q_batches) * 1e3, 2),
                "launches_timed": KERNEL_BATCHES * KERNEL_BATCH_LAUNCHES, "batches": KERNEL_BATCHES,
                "in_step_probe_us": round(in_step_ms * 1e3, 2),
                "algorithmic_bytes_per_launch": quant_kernel_bytes(n),
                "traffic": traffic, "traffic_source": f"profiles/{os.path.basename(TRAFFIC_FILE)} (ncu capture at commit {traffic_commit})"}

    # ---- T2 / T3 of the same workload, cold (rotating sets) and warm (one set, input largely resident in L2)
    def t_of(fn):
        return statistics.median(timed_batches(fn, KERNEL_BATCHES, 40))

    t2 = t_of(lambda i: L.abs_quantize(*qargs[i % n_sets]))
    t3 = t_of(lambda i: L.abs_dequantize(*dargs[i % n_sets]))
    t1_warm = t_of(lambda i: L.abs_quantize_ex(*gargs[0]))
    t2_warm = t_of(lambda i: L.abs_quantize(*qargs[0]))
    out_b = nb_codes + nb_scales
    breakdown = {
        "workload": f"bf16 {rows}x{cols} IF4, median of {KERNEL_BATCHES} batches",
        "T1_quantize_kernel_us": round(q_ms * 1e3, 2), "T1_gbs": round((2 * n + out_b) / q_ms / 1e6, 1),
        "T2_abs_quantize_us": round(t2 * 1e3, 2), "T2_gbs_dram_basis_4N_plus_out": round((4 * n + out_b) / t2 / 1e6, 1),
        "T2_gbs_effective_2N_plus_out": round((2 * n + out_b) / t2 / 1e6, 1),
        "T3_abs_dequantize_us": round(t3 * 1e3, 2), "T3_gbs": round((2 * n + out_b) / t3 / 1e6, 1),
        "warm_l2_T1_us": round(t1_warm * 1e3, 2), "warm_l2_T2_us": round(t2_warm * 1e3, 2),
        "warm_note": "warm = the same buffer set every call (the 64 MiB input mostly stays in the 126 MB L2)"}

    # ---- the "and larger" half of the target: the same three figures at 16384x8192 (seeded device-side mixture
    # of the format-sweep configuration's recipe: 70 % N(0,1), 30 % Laplace(0,1), 0.1 % of entries x100)
    large = None
    if not args.no_large:
        lr, lc = 16384, 8192
        ln = lr * lc
        gen = torch.Generator(device=dev).manual_seed(6 + 1000 * rank)
        lsets = 4                                             # 4 x 256 MiB of inputs = 8x L2
        lx = []
        for k in range(lsets):
            u = torch.rand((lr, lc), device=dev, generator=gen)
            v = torch.randn((lr, lc), device=dev, generator=gen)
            e = torch.empty((lr, lc), device=dev).exponential_(generator=gen)
            sgn = torch.where(torch.rand((lr, lc), device=dev, generator=gen) < 0.5, -1.0, 1.0)
            v = torch.where(u < 0.7, v, e * sgn)
            v = torch.where(torch.rand((lr, lc), device=dev, generator=gen) < 0.001, v * 100.0, v)
            lx.append(v.to(torch.bfloat16))
            del u, v, e, sgn
        lcb, lsb = B.abs_codes_bytes(FMT_IF4, lr, lc), B.abs_scales_bytes(FMT_IF4, lr, lc)
        lcodes = [torch.empty(lcb, dtype=torch.uint8, device=dev) for _ in range(lsets)]
        lscales = [torch.empty(lsb, dtype=torch.uint8, device=dev) for _ in range(lsets)]
        lalpha = [torch.zeros(1, dtype=torch.float32, device=dev) for _ in range(lsets)]
        lout = [torch.empty((lr, lc), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        lq = [(FMT_IF4, lx[k].data_ptr(), lr, lc, lcodes[k].data_ptr(), lscales[k].data_ptr(), lalpha[k].data_ptr(), sp)
              for k in range(lsets)]
        lg = [a[:-1] + (C.byref(og), sp) for a in lq]
        ld = [(FMT_IF4, lcodes[k].data_ptr(), lscales[k].data_ptr(), lalpha[k].data_ptr(), lr, lc,
               lout[k % 2].data_ptr(), sp) for k in range(lsets)]
        for k in range(lsets):
            L.abs_quantize(*lq[k])
        lt2 = statistics.median(timed_batches(lambda i: L.abs_quantize(*lq[i % lsets]), KERNEL_BATCHES, 24, warm=4))
        lt1 = statistics.median(timed_batches(lambda i: L.abs_quantize_ex(*lg[i % lsets]), KERNEL_BATCHES, 24, warm=4))
        lt3 = statistics.median(timed_batches(lambda i: L.abs_dequantize(*ld[i % lsets]), KERNEL_BATCHES, 24, warm=4))
        lob = lcb + lsb
        large = {"workload": f"bf16 {lr}x{lc} IF4 (format-sweep mixture, generated on the device, seed 6), "
                             f"median of {KERNEL_BATCHES} batches of 24 calls, {lsets} rotating sets",
                 "T1_quantize_kernel_us": round(lt1 * 1e3, 2), "T1_gbs": round((2 * ln + lob) / lt1 / 1e6, 1),
                 "T1_frac_of_measured_peak": round((2 * ln + lob) / lt1 / 1e6 / peak, 4),
                 "T2_abs_quantize_us": round(lt2 * 1e3, 2),
                 "T2_gbs_dram_basis_4N_plus_out": round((4 * ln + lob) / lt2 / 1e6, 1),
                 "T2_gbs_effective_2N_plus_out": round((2 * ln + lob) / lt2 / 1e6, 1),
                 "T3_abs_dequantize_us": round(lt3 * 1e3, 2), "T3_gbs": round((2 * ln + lob) / lt3 / 1e6, 1)}
        del lx, lcodes, lscales, lout

    # ---- the matrix product of two IF4 operands with the MAC arithmetic of Sec. 5.2 (abs_matmul, tcgen05): the one
    # dense contraction of the library, so its roofline is the tensor one.  Nine block-scaled FP4 MMAs are issued per
    # useful one; `achieved` counts the MMAs issued.  No FP4 peak was measured on this machine: the denominator is the
    # measured bf16 rate x 4 (the nominal FP4 : bf16 ratio).
    matmul = None
    if not args.no_matmul:
        mm = 4096
        gen = torch.Generator(device=dev).manual_seed(11 + 1000 * rank)
        ma = torch.randn((mm, mm), device=dev, generator=gen).to(torch.bfloat16)
        mb = (torch.randn((mm, mm), device=dev, generator=gen) * 0.02).to(torch.bfloat16)
        qa, qb = B.abs_quantize(FMT_IF4, ma), B.abs_quantize(FMT_IF4, mb)
        mws = torch.empty(L.abs_matmul_workspace_bytes(FMT_IF4, mm, mm, mm) + 1024, dtype=torch.uint8, device=dev)
        mout = torch.empty((mm, mm), dtype=torch.float32, device=dev)
        B.abs_matmul(FMT_IF4, qa, qb, mm, mm, mm, out=mout, workspace=mws, check=True)
        mt = statistics.median(timed_batches(lambda i: B.abs_matmul(FMT_IF4, qa, qb, mm, mm, mm, out=mout, workspace=mws),
                                             KERNEL_BATCHES, 20, warm=4))
        tpeak, tsrc = bf16_tensor_peak()
        issued = 9 * 2 * mm ** 3 / (mt * 1e-3) / 1e12
        matmul = {"workload": f"IF4 x IF4, {mm}^3, N(0,1) x N(0,0.02), operand split + product per call, "
                              f"median of {KERNEL_BATCHES} batches of 20 calls",
                  "ms_per_call": round(mt, 4), "useful_tflops": round(issued / 9, 1),
                  "roofline": {"bound": "tensor", "achieved": round(issued, 1), "peak": round(4 * tpeak, 1),
                               "unit": "TFLOP/s", "frac": round(issued / (4 * tpeak), 4),
                               "peak_source": tsrc + " x 4 (nominal FP4 : bf16)",
                               "frac_of_nominal_9000_tflops": round(issued / 9000.0, 4),
                               "flops_counted": "the nine block-scaled FP4 MMAs issued per useful one"}}
        del ma, mb, qa, qb, mws, mout

    # ---- for information: the same result through the one-pass emulation call (amax pass + one kernel that
    # quantizes and decodes from registers, writing codes, scales and the bf16 output); not part of `value`.
    eargs = [(FMT_IF4, xs[k].data_ptr(), rows, cols, outs[k].data_ptr(), codes[k].data_ptr(), scales[k].data_ptr(),
              alphas[k].data_ptr(), None, sp) for k in range(n_sets)]
    e_ms = t_of(lambda i: L.abs_quantize_dequantize(*eargs[i % n_sets]))
    one_pass = {"us_per_call": round(e_ms * 1e3, 2), "calls_timed": KERNEL_BATCHES * 40,
                "api": "abs_quantize_dequantize with code outputs (same outputs as one step, 2 kernels instead of 3)"}

    # ---- for information: the same steps issued alternately on two streams, so the bandwidth-bound amax /
    # dequantize kernels of one tensor overlap the issue-bound group-quantize kernel of another (independent
    # tensors, as in a layer with several operands to quantize); not part of `value`.
    s2 = [torch.cuda.Stream(device=dev) for _ in range(2)]
    sp2 = [C.c_void_p(s.cuda_stream) for s in s2]

    def step2(i):
        k, p = i % n_sets, sp2[i & 1]
        L.abs_quantize(*qargs[k][:-1], p)
        L.abs_dequantize(*dargs[k][:-1], p)

    n_t = 200
    for i in range(4):
        step2(i)
    torch.cuda.synchronize()
    t0e, t1e, j = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True), torch.cuda.Event())
    t0e.record(s2[0])
    s2[1].wait_event(t0e)
    for i in range(n_t):
        step2(i)
    j.record(s2[1])
    s2[0].wait_event(j)
    t1e.record(s2[0])
    torch.cuda.synchronize()
    t_us = t0e.elapsed_time(t1e) / n_t * 1e3
    two_streams = {"us_per_step": round(t_us, 2), "value": round(step_bytes(n) / (t_us * 1e-6) / 1e9, 1),
                   "unit": UNIT, "steps_timed": n_t,
                   "note": "steps alternate over two streams; per-rank figure, informational"}
    sampler.stop()

    # ---- end to end through the host-buffer C-ABI calls (pinned host memory, copies in the timed region)
    e2e_steps = 0 if args.no_e2e else max(1, min(args.steps, 20))
    ws = torch.empty(B.abs_host_workspace_bytes(FMT_IF4, rows, cols), dtype=torch.uint8, device=dev)
    xh = torch.from_numpy(xb.view(np.int16)).pin_memory()
    ch = torch.empty(nb_codes, dtype=torch.uint8).pin_memory()
    sh = torch.empty(nb_scales, dtype=torch.uint8).pin_memory()
    ah = torch.zeros(1, dtype=torch.float32).pin_memory()
    oh = torch.empty((rows, cols), dtype=torch.int16).pin_memory()

    def e2e_step():
        B.abs_quantize_host(FMT_IF4, xh, ch, sh, ah, ws)
        B.abs_dequantize_host(FMT_IF4, ch, sh, ah, rows, cols, oh, ws)

    for _ in range(3 if e2e_steps else 0):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = (time.perf_counter() - t0) / max(e2e_steps, 1)
    t = torch.tensor([e2e_s], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    e2e_s = float(t.item())
    e2e = {"value": round(world * step_bytes(n) / e2e_s / 1e9, 2) if e2e_steps else None, "unit": UNIT,
           "h2d_bytes_per_step": 2 * n + nb_codes + nb_scales + 4, "d2h_bytes_per_step": nb_codes + nb_scales + 4 + 2 * n,
           "ms_per_step": round(e2e_s * 1e3, 3), "steps": e2e_steps,
           "api": "abs_quantize_host + abs_dequantize_host (pinned host buffers)"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{WORKLOAD}: IF4 quantize+dequantize, bf16 {rows}x{cols}, {cfg.note}",
                       "data_dtype": "bf16 in and out, FP32 arithmetic, 4-bit codes + E4M3 scales",
                       "bytes_per_step": step_bytes(n), "elements_per_s": round(world * n / (ms_per_step * 1e-3), 0),
                       "l2": f"cold: steps rotate over {n_sets} buffer sets; the inputs alone are "
                             f"{n_sets * 2 * n >> 20} MiB >= 4x L2, all buffers {n_sets * set_bytes >> 20} MiB",
                       "sharding": "one independent tensor per rank, no collective",
                       "input_sha256": I.sha256(xb)[:16]},
            "clock_ramp_ms": round(clock_ramp_ms, 1), "clock_ramp_steps": ramp_steps,
            "ms_per_step_batches": {"median": round(statistics.median(step_batches), 5),
                                    "best": round(min(step_batches), 5), "worst": round(max(step_batches), 5),
                                    "batches": KERNEL_BATCHES, "steps_per_batch": KERNEL_BATCH_LAUNCHES},
            "roofline": roofline, "breakdown": breakdown, "large": large, "matmul": matmul,
            "e2e": e2e, "one_pass": one_pass, "two_streams": two_streams,
            "gpu_launches": 3 * args.steps,
            "clocks": clocks,
        }
        if world == 1 and not args.no_cpu_baseline:
            threads = os.cpu_count() or 1
            gbs, best = oracle_rate(xb, 3, threads)
            line["cpu_baseline"] = {"value": round(gbs, 4), "unit": UNIT, "cores": threads, "kind": "oracle",
                                    "sample": f"the whole {rows}x{cols} tensor, quantize+dequantize, best of 3 "
                                              f"({best:.3f} s), {threads} threads over rows"}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["cuda", "reference"], default="cuda")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiling runs)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-ramp", action="store_true", help="skip the clock-ramp loop (profiling runs only: fewer launches)")
    ap.add_argument("--no-large", action="store_true", help="skip the 16384x8192 figures (profiling runs)")
    ap.add_argument("--no-matmul", action="store_true", help="skip the abs_matmul figure (profiling runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()

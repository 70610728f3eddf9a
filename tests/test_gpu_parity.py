"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, bit for bit.

Codes, scale bytes (selection bit included), alpha and dequantized outputs must be identical
on the same seeded inputs: integer / byte work is compared exactly, and the floating-point
outputs (alpha, dequantized bf16 / fp32) are compared by bit pattern too, because both sides
fix the same FP32 operation order.
"""
import os

import numpy as np
import pytest

from paper_2603_28765_b200 import inputs as I

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
THREADS = max(1, min(32, os.cpu_count() or 1))
ALL_FMTS = [0, 1, 2, 3, 4, 5, 6, 7]          # 5..7: the block-size-8 variants


@pytest.fixture(scope="module")
def B():
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    from paper_2603_28765_b200 import binding
    binding.lib()          # raises if the CUDA library is missing: there is no fallback
    return binding


def to_dev(xb: np.ndarray):
    return torch.from_numpy(xb.view(np.int16)).cuda().view(torch.bfloat16)


def gpu_quantize(B, fmt, xb, flags=0, mask=0, seed=0, alpha=None):
    x = to_dev(xb)
    opts = B.make_opts(flags, mask, seed)
    ts = None
    if flags & B.ABS_F_ALPHA_GIVEN:
        ts = torch.tensor([alpha], dtype=torch.float32, device="cuda")
    codes, scales, ts = B.abs_quantize(fmt, x, tensor_scale=ts, opts=opts)
    torch.cuda.synchronize()
    rows, cols = xb.shape
    nb = rows * cols * B.FMT_BITS[fmt] // 8
    return (codes[:nb].cpu().numpy().reshape(rows, -1) if nb else np.zeros((rows, 0), np.uint8),
            scales[:rows * cols // B.FMT_GROUP[fmt]].cpu().numpy().reshape(rows, -1) if nb else np.zeros((rows, 0), np.uint8),
            np.float32(ts.item()), (codes, scales, ts))


def assert_same(name, got, want):
    got = np.asarray(got)
    want = np.asarray(want)
    assert got.shape == want.shape, (name, got.shape, want.shape)
    if not np.array_equal(got, want):
        bad = np.argwhere(got != want)
        raise AssertionError(f"{name}: {len(bad)} of {got.size} differ; first at {bad[:5].tolist()} "
                             f"got {got[tuple(bad[0])]} want {want[tuple(bad[0])]}")


def check_case(B, oracle, fmt, xb, flags=0, mask=0, seed=0, alpha=None, dequant=True):
    rows, cols = xb.shape
    c, s, a, dev = gpu_quantize(B, fmt, xb, flags, mask, seed, alpha)
    oc, osc, oa = oracle.quantize(fmt, xb, flags=flags, sign_mask=mask, sr_seed=seed, alpha=alpha, threads=THREADS)
    assert np.float32(a).view(np.uint32) == np.float32(oa).view(np.uint32), ("alpha", a, oa)
    assert_same("scales", s, osc)
    assert_same("codes", c, oc)
    if dequant and rows * cols:
        out = B.abs_dequantize(fmt, dev[0], dev[1], dev[2], rows, cols)
        want = oracle.dequantize(fmt, oc, osc, oa, rows, cols, threads=THREADS)
        assert_same("dequant bf16", out.view(torch.int16).cpu().numpy().view(np.uint16), want)
        out32 = B.abs_dequantize(fmt, dev[0], dev[1], dev[2], rows, cols, opts=B.make_opts(B.ABS_F_OUT_FP32))
        want32 = oracle.dequantize(fmt, oc, osc, oa, rows, cols, out_fp32=True, threads=THREADS)
        assert_same("dequant fp32", out32.cpu().numpy().view(np.uint32), want32.view(np.uint32))
    return s


# ------------------------------------------------------------------ the converts the kernels rely on

@pytest.mark.parametrize("kind,fmt", [(0, None), (1, 1), (2, 2), (3, 3), (4, 4)])
def test_hardware_converts_match_oracle_exhaustively(B, oracle, kind, fmt):
    """All 2^32 FP32 inputs go through the device convert; the output is checked to be monotone in
    |x| on the device, and every change point (plus its neighbour) is compared with the oracle, which
    is monotone by construction -- together that is equality on every finite input."""
    enc = (lambda v: oracle.e4m3_encode(v)) if kind == 0 else (lambda v: oracle.fp_encode(fmt, v))
    chunk = 1 << 28
    top_finite = 0x7F800000
    for sign in (0, 1):
        if kind == 0 and sign == 1:
            continue          # scale inputs are non-negative
        prev_last = None
        changes = []
        for start in range(0, top_finite, chunk):
            n = min(chunk, top_finite - start)
            bits = torch.arange(start, start + n, dtype=torch.int32, device="cuda")
            if sign:
                bits = bits + (-2 ** 31)          # sets the sign bit of the pattern
            f = bits.view(torch.float32)
            out = B.abs_selftest_convert(kind, f)
            o = out.to(torch.int16)
            d = o[1:] - o[:-1]
            assert int(d.min()) >= 0, "device convert is not monotone in |x|"
            idx = torch.nonzero(d).flatten().cpu().numpy()
            ocpu = out[idx + 1].cpu().numpy() if len(idx) else np.zeros(0, np.uint8)
            for i, code in zip(idx, ocpu):
                changes.append((start + int(i) + 1, int(code)))
            first, last = int(out[0]), int(out[-1])
            if prev_last is not None and first != prev_last:
                assert first > prev_last
                changes.append((start, first))
            elif prev_last is None:
                changes.append((start, first))
            prev_last = last
            del bits, f, out, o, d
        assert len(changes) >= 4
        for pos, code in changes:
            v = np.array([pos | (sign << 31)], dtype=np.uint32).view(np.float32)[0]
            assert enc(v) == code, (kind, hex(pos), code, enc(v))
            if pos > 0:
                vm = np.array([(pos - 1) | (sign << 31)], dtype=np.uint32).view(np.float32)[0]
                assert enc(vm) < code
        # +-inf saturate like the largest finite input
        vinf = torch.tensor([np.inf if sign == 0 else -np.inf], dtype=torch.float32, device="cuda")
        assert int(B.abs_selftest_convert(kind, vinf)[0]) == enc(np.float32(np.inf if sign == 0 else -np.inf))


@pytest.mark.parametrize("k,fmt", [(0, None), (1, 1), (2, 2), (3, 3), (4, 4)])
def test_device_decode_tables(B, oracle, k, fmt):
    n = 127 if k == 0 else (1 << B.FMT_BITS[fmt])
    codes = torch.arange(n, dtype=torch.float32, device="cuda")
    got = B.abs_selftest_convert(16 + k, codes).cpu().numpy()
    want = np.array([oracle.e4m3_value(c) if k == 0 else oracle.fp_value(fmt, c) for c in range(n)], dtype=np.float32)
    assert_same("decode", got.view(np.uint32), want.view(np.uint32))


def test_device_rint_is_ties_even(B):
    v = torch.tensor([0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 6.5, 7.4999995, -7.5, 30.5, 31.5], dtype=torch.float32,
                     device="cuda")
    got = B.abs_selftest_convert(5, v).cpu().numpy().astype(np.int8)
    assert list(got) == [0, 2, 2, 0, -2, -2, 6, 7, -8, 30, 32]


# ------------------------------------------------------------------ parity on the configurations

SMALL = {
    "cfg1": ("cfg1", 256, 1024),            # the full first configuration
    "cfg2": ("cfg2", 300, 4096),            # several tiles and a ragged tail (300 rows)
    "cfg3a": ("cfg3a", 64, 14336),
    "cfg3b": ("cfg3b", 515, 4096),
    "cfg4": ("cfg4", 384, 8192),
    "cfg5": ("cfg5", 257, 8192),
}


@pytest.mark.parametrize("fmt", ALL_FMTS)
@pytest.mark.parametrize("case", sorted(SMALL))
def test_rtn_parity_small(B, oracle, fmt, case):
    name, rows, cols = SMALL[case]
    check_case(B, oracle, fmt, I.generate(name, rows, cols))


@pytest.mark.parametrize("fmt", ALL_FMTS)
@pytest.mark.parametrize("case", sorted(I.edge_tensors()))
def test_edge_tensor_parity(B, oracle, fmt, case):
    check_case(B, oracle, fmt, I.edge_tensors()[case])


@pytest.mark.parametrize("fmt", ALL_FMTS)
@pytest.mark.parametrize("flags", ["H", "S", "S17", "HS", "HS17"])
def test_option_parity(B, oracle, fmt, flags):
    f = (B.ABS_F_HADAMARD16 if "H" in flags else 0) | (B.ABS_F_STOCHASTIC if "S" in flags else 0) \
        | (B.ABS_F_SR_SCALE_17_16 if "17" in flags else 0)
    mask = oracle.hadamard_sign_mask(2024)
    for name, rows, cols in (("cfg4", 200, 2048), ("cfg2", 96, 1024), ("cfg1", 64, 256)):
        check_case(B, oracle, fmt, I.generate(name, rows, cols), flags=f, mask=mask, seed=0xDEADBEEF12345678)
    for case in ("tiny_row", "wide_dynamic_range", "signed_zeros", "zeros_3x48", "ragged_37x208"):
        check_case(B, oracle, fmt, I.edge_tensors()[case], flags=f, mask=mask, seed=99)


def test_sr_stream_depends_on_the_seed_only(B, oracle):
    """Different seeds give different streams; the same seed repeats exactly."""
    xb = I.generate("cfg1", 64, 256)
    a = gpu_quantize(B, 1, xb, B.ABS_F_STOCHASTIC, 0, 5)
    b = gpu_quantize(B, 1, xb, B.ABS_F_STOCHASTIC, 0, 5)
    c = gpu_quantize(B, 1, xb, B.ABS_F_STOCHASTIC, 0, 6)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert not np.array_equal(a[0], c[0])


@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_alpha_given_and_worked_example(B, oracle, fmt):
    x = np.zeros((1, 16), np.float32)
    x[0, :4] = [6, 18, 36, 42]
    xb = I.f32_to_bf16_bits(x)
    check_case(B, oracle, fmt, xb, flags=B.ABS_F_ALPHA_GIVEN, alpha=1.0)
    check_case(B, oracle, fmt, xb)
    check_case(B, oracle, fmt, I.generate("cfg5", 64, 512), flags=B.ABS_F_ALPHA_GIVEN, alpha=0.01)
    if fmt == 1:    # Fig. 3a: integer candidate selected, bytes 31 76, scale 0xFE with Eq. 1's alpha
        c, s, a, _ = gpu_quantize(B, 1, xb)
        assert c[0].tobytes() == bytes([0x31, 0x76, 0, 0, 0, 0, 0, 0]) and s[0, 0] == 0xFE and a == np.float32(2 ** -6)


def test_index64_kernel_instances(B, oracle):
    """The 64-bit-index instances (normally chosen beyond 2^31 groups) give the same bytes."""
    xb = I.generate("cfg2", 130, 2048)
    for fmt in (0, 1):
        check_case(B, oracle, fmt, xb, flags=B.ABS_F_INDEX64, dequant=False)
        c, s, a, dev = gpu_quantize(B, fmt, xb)
        out = B.abs_dequantize(fmt, dev[0], dev[1], dev[2], *xb.shape, opts=B.make_opts(B.ABS_F_INDEX64))
        want = oracle.dequantize(fmt, c, s, a, *xb.shape)
        assert_same("dequant", out.view(torch.int16).cpu().numpy().view(np.uint16), want)
    # an input that is only 16-byte aligned takes the two-128-bit-access path
    buf = torch.zeros(130 * 2048 + 8, dtype=torch.bfloat16, device="cuda")
    x = buf[8:].view(130, 2048)
    x.copy_(to_dev(xb))
    assert x.data_ptr() % 32 == 16
    codes, scales, ts = B.abs_quantize(1, x)
    oc, osc, oa = oracle.quantize(1, xb)
    assert_same("codes", codes.cpu().numpy().reshape(130, -1), oc)
    assert_same("scales", scales.cpu().numpy().reshape(130, -1), osc)
    obuf = torch.zeros(130 * 2048 + 8, dtype=torch.bfloat16, device="cuda")
    out = B.abs_dequantize(1, codes, scales, ts, 130, 2048, out=obuf[8:].view(130, 2048))
    assert_same("dequant", out.view(torch.int16).cpu().numpy().view(np.uint16), oracle.dequantize(1, oc, osc, oa, 130, 2048))


def test_large_tensor_sampled_parity(B, oracle):
    """2.6e9 elements (5.2 GB of bf16: byte offsets and element indices beyond 2^32 / 2^31), in the
    launch configuration the library picks itself.  alpha is checked against torch's max; 48 sampled
    rows plus the first and last are compared with the oracle byte for byte (quantize with the
    stochastic option too, whose random stream is indexed by the element position)."""
    rows, cols = 40000, 65536
    g = torch.Generator(device="cuda").manual_seed(11)
    block = torch.randn(500, cols, device="cuda", generator=g)
    x = torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda")
    for r0 in range(0, rows, 500):
        scale = 0.25 + 4 * torch.rand(500, 1, device="cuda", generator=g)
        x[r0:r0 + 500] = (block * scale).to(torch.bfloat16)
    x[rows - 3, cols - 5] = 77.0                                  # the maximum sits near the end
    del block
    amax = float(x.abs().max().float().item())
    pick = sorted(set([0, rows - 1, rows - 3] + [int(v) for v in np.random.default_rng(3).integers(0, rows, 48)]))
    xs = x[pick].contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    for fmt, flags in ((1, 0), (1, B.ABS_F_STOCHASTIC), (0, 0)):
        codes, scales, ts = B.abs_quantize(fmt, x, opts=B.make_opts(flags, 0, 99))
        torch.cuda.synchronize()
        alpha = oracle.alpha_from_amax(fmt, np.float32(amax))
        assert np.float32(ts.item()).view(np.uint32) == np.float32(alpha).view(np.uint32)
        cg = codes.view(rows, cols // 2)[pick].cpu().numpy()
        sg = scales.view(rows, cols // 16)[pick].cpu().numpy()
        for i, r in enumerate(pick):
            if flags & B.ABS_F_STOCHASTIC:
                # the oracle indexes the random stream by row * cols + col: give it the row offset by
                # quantizing a tensor view that starts at row r (rows before it are never touched)
                oc, osc = oracle_rows_with_offset(oracle, fmt, xs[i:i + 1], r, cols, alpha, flags, 99)
            else:
                oc, osc, _ = oracle.quantize(fmt, xs[i:i + 1], flags=B.ABS_F_ALPHA_GIVEN, alpha=alpha)
            assert_same(f"codes row {r}", cg[i:i + 1], oc)
            assert_same(f"scales row {r}", sg[i:i + 1], osc)
        if flags == 0:
            out = B.abs_dequantize(fmt, codes, scales, ts, rows, cols)
            og = out[pick].view(torch.int16).cpu().numpy().view(np.uint16)
            for i, r in enumerate(pick):
                oc, osc, _ = oracle.quantize(fmt, xs[i:i + 1], flags=B.ABS_F_ALPHA_GIVEN, alpha=alpha)
                assert_same(f"dequant row {r}", og[i:i + 1], oracle.dequantize(fmt, oc, osc, alpha, 1, cols))
            del out
        del codes, scales


def oracle_rows_with_offset(oracle, fmt, row_bits, row_index, cols, alpha, flags, seed):
    """Oracle result for one row that sits at `row_index` of a larger tensor (matters only for the
    element index of the stochastic stream)."""
    c, s, _ = oracle.quantize(fmt, np.ascontiguousarray(row_bits), flags=flags | oracle.F_ALPHA_GIVEN, alpha=alpha,
                              sr_seed=seed, sr_index_offset=int(row_index) * cols)
    return c, s


def test_amax_entry_point(B, oracle):
    xb = I.generate("cfg2", 123, 2048)
    mask = 0x5A3C
    for flags in (0, B.ABS_F_HADAMARD16):
        got = B.abs_amax(to_dev(xb), opts=B.make_opts(flags, mask)).item()
        want = oracle.amax(xb, flags=flags, sign_mask=mask, threads=THREADS)
        assert np.float32(got).view(np.uint32) == np.float32(want).view(np.uint32)
        for fmt in ALL_FMTS:
            a = np.float32(B.abs_alpha_from_amax(fmt, float(want)))
            assert a.view(np.uint32) == np.float32(oracle.alpha_from_amax(fmt, want)).view(np.uint32)


def test_back_to_back_calls_reuse_scratch(B, oracle):
    """The amax scratch slot re-arms itself: many calls in a row, on two streams, stay exact."""
    xs = [I.generate("cfg1", 64, 256, seed=s) for s in range(4)]
    want = [oracle.quantize(1, x) for x in xs]
    devs = [to_dev(x) for x in xs]
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs = []
    for rep in range(600):      # wraps the scratch ring more than once across both streams
        k = rep % 4
        outs.append((k, B.abs_quantize(1, devs[k], stream=(s1 if rep % 2 else s2))))
    torch.cuda.synchronize()
    for k, (c, s, a) in outs[-16:]:
        assert np.float32(a.item()) == want[k][2]
        assert np.array_equal(c.cpu().numpy().reshape(64, -1), want[k][0])
        assert np.array_equal(s.cpu().numpy().reshape(64, -1), want[k][1])


@pytest.mark.parametrize("rows", [48, 96, 1000])
def test_host_buffer_entry_points(B, oracle, rows):
    """Host-buffer calls; from 64 rows on abs_dequantize_host works in row chunks on two streams (the last
    chunk of 1000 rows is shorter than the others)."""
    xb = I.generate("cfg5", rows, 1024)
    rows, cols = xb.shape
    for fmt in ALL_FMTS:
        ws = torch.empty(B.abs_host_workspace_bytes(fmt, rows, cols), dtype=torch.uint8, device="cuda")
        xh = torch.from_numpy(xb.view(np.int16)).pin_memory()
        ch = torch.empty(B.abs_codes_bytes(fmt, rows, cols), dtype=torch.uint8).pin_memory()
        sh = torch.empty(B.abs_scales_bytes(fmt, rows, cols), dtype=torch.uint8).pin_memory()
        ah = torch.zeros(1, dtype=torch.float32).pin_memory()
        B.abs_quantize_host(fmt, xh, ch, sh, ah, ws)
        oc, osc, oa = oracle.quantize(fmt, xb)
        assert np.float32(ah.item()) == oa
        assert_same("codes", ch.numpy().reshape(rows, -1), oc)
        assert_same("scales", sh.numpy().reshape(rows, -1), osc)
        oh = torch.empty((rows, cols), dtype=torch.int16).pin_memory()
        B.abs_dequantize_host(fmt, ch, sh, ah, rows, cols, oh, ws)
        assert_same("dequant", oh.numpy().view(np.uint16), oracle.dequantize(fmt, oc, osc, oa, rows, cols))


def test_argument_validation_on_device(B):
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    L = B.lib()
    codes = torch.zeros(256, dtype=torch.uint8, device="cuda")
    scales = torch.zeros(64, dtype=torch.uint8, device="cuda")
    ts = torch.zeros(4, dtype=torch.float32, device="cuda")
    q = lambda fmt, xp, r, c, cp, sp, tp, o=None: L.abs_quantize_ex(fmt, xp, r, c, cp, sp, tp, o, None)
    assert q(19, x.data_ptr(), 4, 64, codes.data_ptr(), scales.data_ptr(), ts.data_ptr()) == 4
    assert q(1, x.data_ptr(), 4, 60, codes.data_ptr(), scales.data_ptr(), ts.data_ptr()) == 2
    assert q(1, x.data_ptr(), -1, 64, codes.data_ptr(), scales.data_ptr(), ts.data_ptr()) == 2
    assert q(1, None, 4, 64, codes.data_ptr(), scales.data_ptr(), ts.data_ptr()) == 1
    assert q(1, x.data_ptr() + 2, 4, 64, codes.data_ptr(), scales.data_ptr(), ts.data_ptr()) == 3
    import ctypes
    bad = B.make_opts(1 << 9)
    assert q(1, x.data_ptr(), 4, 64, codes.data_ptr(), scales.data_ptr(), ts.data_ptr(), ctypes.byref(bad)) == 5
    assert q(1, x.data_ptr(), 0, 64, codes.data_ptr(), scales.data_ptr(), ts.data_ptr()) == 0
    sr = B.make_opts(B.ABS_F_STOCHASTIC)
    assert L.abs_dequantize_ex(1, codes.data_ptr(), scales.data_ptr(), ts.data_ptr(), 4, 64, x.data_ptr(),
                               ctypes.byref(sr), None) == 5
    torch.cuda.synchronize()


@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_input_aligned_to_16_but_not_32_bytes(B, oracle, fmt):
    """The kernels use 256-bit loads when the input allows it; a tensor that starts 16 bytes into an
    allocation takes their 128-bit fallbacks (plain, Hadamard + stochastic rounding, amax)."""
    xb = I.generate("cfg2", 70, 1024)
    rows, cols = xb.shape
    buf = torch.zeros(rows * cols + 8, dtype=torch.bfloat16, device="cuda")
    assert buf.data_ptr() % 32 == 0
    x = buf[8:].view(rows, cols)
    x.copy_(to_dev(xb))
    assert x.data_ptr() % 32 == 16
    mask = oracle.hadamard_sign_mask(5)
    for flags in (0, B.ABS_F_HADAMARD16 | B.ABS_F_STOCHASTIC | B.ABS_F_SR_SCALE_17_16):
        codes, scales, ts = B.abs_quantize(fmt, x, opts=B.make_opts(flags, mask, 1234))
        torch.cuda.synchronize()
        oc, os_, oa = oracle.quantize(fmt, xb, flags=flags, sign_mask=mask, sr_seed=1234)
        assert np.float32(ts.item()) == oa
        assert_same("codes", codes.cpu().numpy()[:oc.size].reshape(oc.shape), oc)
        assert_same("scales", scales.cpu().numpy()[:os_.size].reshape(os_.shape), os_)


def test_guard_bands_stay_untouched(B, oracle):
    """Outputs are written inside their buffers only: sentinel bytes around them survive."""
    for fmt in ALL_FMTS:
        xb = I.generate("cfg1", 37, 208)
        rows, cols = xb.shape
        nb, ns = B.abs_codes_bytes(fmt, rows, cols), B.abs_scales_bytes(fmt, rows, cols)
        pad = 256
        cbuf = torch.full((nb + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda")
        sbuf = torch.full((ns + 2 * pad + 15,), 0xA5, dtype=torch.uint8, device="cuda")
        obuf = torch.full((rows * cols * 2 + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda")
        codes, scales, out = cbuf[pad:pad + nb], sbuf[pad:pad + ns], obuf[pad:pad + rows * cols * 2]
        ts = torch.zeros(1, dtype=torch.float32, device="cuda")
        B.abs_quantize(fmt, to_dev(xb), codes=codes, scales=scales, tensor_scale=ts)
        B.abs_dequantize(fmt, codes, scales, ts, rows, cols, out=out.view(torch.bfloat16).view(rows, cols))
        torch.cuda.synchronize()
        for buf, n in ((cbuf, nb), (sbuf, ns), (obuf, rows * cols * 2)):
            assert bool((buf[:pad] == 0xA5).all()) and bool((buf[pad + n:] == 0xA5).all())


# ------------------------------------------------------------------ full-size configurations

FULL = [
    ("cfg2", [1], 0),
    ("cfg3a", [0, 1], 0),
    ("cfg3b", [0, 1], 0),
    ("cfg5", [0, 1, 2, 3, 4, 5, 6, 7], 0),
    ("cfg4", [1], "HS17"),
    ("cfg4", [0], "HS17"),
]


@pytest.mark.parametrize("name,fmts,opt", FULL, ids=[f"{f[0]}-{''.join(map(str, f[1]))}" for f in FULL])
def test_full_size_parity(B, oracle, name, fmts, opt):
    """Element-by-element comparison at the benchmark's full sizes (the oracle, threaded over rows,
    still finishes in seconds per format)."""
    xb = I.generate(name)
    flags, mask, seed = 0, 0, 0
    if opt == "HS17":
        flags = B.ABS_F_HADAMARD16 | B.ABS_F_STOCHASTIC | B.ABS_F_SR_SCALE_17_16
        mask, seed = oracle.hadamard_sign_mask(5), 5
    for fmt in fmts:
        s = check_case(B, oracle, fmt, xb, flags=flags, mask=mask, seed=seed)
        if fmt not in (0, 5):
            frac = float((s >> 7).mean())
            assert 0.05 < frac < 0.999, (name, fmt, frac)
    if opt == "HS17" and 1 in fmts:       # the extra row of the gradient configuration: 17/16 option off
        check_case(B, oracle, 1, xb, flags=flags & ~B.ABS_F_SR_SCALE_17_16, mask=mask, seed=seed, dequant=False)


def test_sr_bias_signature_on_gpu(B):
    """App. B on the CUDA path: averaged over seeds, NVFP4 with stochastic rounding leaves every
    magnitude bin unchanged, IF4 moves the near-maximal values of a group outward, by well under
    5 % of the group maximum, and only a small share of the elements sits in the affected bins."""
    from paper_2603_28765_b200 import sr_bias
    res = sr_bias.run(trials=200, rows=256, cols=4096, scale_option=True)
    nv = {round(b["rel_lo"], 1): b for b in res["nvfp4"]}
    i4 = {round(b["rel_lo"], 1): b for b in res["if4"]}
    for lo, b in nv.items():
        assert abs(b["mean_change_over_gmax"]) < 3e-3, ("nvfp4", lo, b)
    top = i4[0.9]
    assert 3e-3 < top["mean_change_over_gmax"] < 5e-2, top
    assert top["share"] < 0.12
    for lo in (0.1, 0.2, 0.3, 0.4):
        assert abs(i4[lo]["mean_change_over_gmax"]) < 6e-3, (lo, i4[lo])


@pytest.mark.parametrize("fmt", [0, 1])
def test_transposed_quantize_equals_quantize_of_transpose(B, oracle, fmt):
    """abs_quantize_transposed(X) must give the bytes the oracle gives for X^T (the plain definition),
    on shapes with several column tiles, a ragged last tile and many row blocks; dequantizing with
    swapped dimensions returns the transposed matrix's dequantization."""
    for name, rows, cols in (("cfg2", 304, 4096), ("cfg3a", 64, 14336), ("cfg5", 2048, 1040), ("cfg1", 16, 16)):
        xb = I.generate(name, rows, cols)
        xt = np.ascontiguousarray(xb.T)
        ct, st, ts = B.abs_quantize_transposed(fmt, to_dev(xb))
        torch.cuda.synchronize()
        oc, osc, oa = oracle.quantize(fmt, xt, threads=THREADS)
        assert np.float32(ts.item()).view(np.uint32) == np.float32(oa).view(np.uint32)
        assert_same("scales_t", st.cpu().numpy().reshape(cols, -1), osc)
        assert_same("codes_t", ct.cpu().numpy().reshape(cols, -1), oc)
        out = B.abs_dequantize(fmt, ct, st, ts, cols, rows)
        assert_same("dequant_t", out.view(torch.int16).cpu().numpy().view(np.uint16),
                    oracle.dequantize(fmt, oc, osc, oa, cols, rows, threads=THREADS))
    # with the Hadamard option (Sec. 4.1: transform, then quantize, both along the token dimension)
    mask = oracle.hadamard_sign_mask(31)
    for name, rows, cols in (("cfg4", 320, 2048), ("cfg2", 64, 528)):
        xb = I.generate(name, rows, cols)
        ct, st, ts = B.abs_quantize_transposed(fmt, to_dev(xb), opts=B.make_opts(B.ABS_F_HADAMARD16, mask))
        torch.cuda.synchronize()
        oc, osc, oa = oracle.quantize(fmt, np.ascontiguousarray(xb.T), flags=oracle.F_HADAMARD16, sign_mask=mask,
                                      threads=THREADS)
        assert np.float32(ts.item()).view(np.uint32) == np.float32(oa).view(np.uint32)
        assert_same("scales_t rht", st.cpu().numpy().reshape(cols, -1), osc)
        assert_same("codes_t rht", ct.cpu().numpy().reshape(cols, -1), oc)
    # the gradient recipe of Sec. 4.1 / App. B along the token dimension: Hadamard, stochastic rounding, 17/16
    for flags in (B.ABS_F_STOCHASTIC, B.ABS_F_HADAMARD16 | B.ABS_F_STOCHASTIC | B.ABS_F_SR_SCALE_17_16):
        for name, rows, cols in (("cfg4", 320, 2048), ("cfg2", 80, 528)):
            xb = I.generate(name, rows, cols)
            ct, st, ts = B.abs_quantize_transposed(fmt, to_dev(xb), opts=B.make_opts(flags, mask, 0xABCDEF0123))
            torch.cuda.synchronize()
            oc, osc, oa = oracle.quantize(fmt, np.ascontiguousarray(xb.T), flags=flags, sign_mask=mask,
                                          sr_seed=0xABCDEF0123, threads=THREADS)
            assert np.float32(ts.item()).view(np.uint32) == np.float32(oa).view(np.uint32)
            assert_same("scales_t sr", st.cpu().numpy().reshape(cols, -1), osc)
            assert_same("codes_t sr", ct.cpu().numpy().reshape(cols, -1), oc)
    # alpha given, and the argument checks
    xb = I.generate("cfg5", 64, 256)
    ts = torch.tensor([0.02], dtype=torch.float32, device="cuda")
    ct, st, _ = B.abs_quantize_transposed(fmt, to_dev(xb), tensor_scale=ts, opts=B.make_opts(B.ABS_F_ALPHA_GIVEN))
    oc, osc, _ = oracle.quantize(fmt, np.ascontiguousarray(xb.T), flags=oracle.F_ALPHA_GIVEN, alpha=0.02)
    assert_same("codes_t", ct.cpu().numpy().reshape(256, -1), oc)
    L = B.lib()
    x = to_dev(xb)
    assert L.abs_quantize_transposed(2, x.data_ptr(), 64, 256, ct.data_ptr(), st.data_ptr(), ts.data_ptr(), None, None) == 4
    assert L.abs_quantize_transposed(1, x.data_ptr(), 40, 256, ct.data_ptr(), st.data_ptr(), ts.data_ptr(), None, None) == 2
    import ctypes
    bad = B.make_opts(B.ABS_F_SCALES_SWIZZLED)
    assert L.abs_quantize_transposed(1, x.data_ptr(), 64, 256, ct.data_ptr(), st.data_ptr(), ts.data_ptr(),
                                     ctypes.byref(bad), None) == 5


@pytest.mark.parametrize("fmt", [0, 1])
def test_fused_quantize_dequantize_is_quantize_then_dequantize(B, oracle, fmt):
    """The one-pass emulation entry point (Sec. 4.1) gives the oracle's quantize followed by its dequantize,
    byte for byte, with and without the optional code outputs, for every option it accepts."""
    mask = oracle.hadamard_sign_mask(9)
    H, S, S17, G = B.ABS_F_HADAMARD16, B.ABS_F_STOCHASTIC, B.ABS_F_SR_SCALE_17_16, B.ABS_F_ALPHA_GIVEN
    for flags in (0, H, S, H | S | S17, G, G | H | S):
        for name, rows, cols in (("cfg2", 300, 1024), ("cfg4", 64, 2064), ("cfg1", 1, 16)):
            xb = I.generate(name, rows, cols)
            alpha = 0.004 if flags & G else None
            ts = torch.tensor([alpha], dtype=torch.float32, device="cuda") if alpha is not None else None
            oc, osc, oa = oracle.quantize(fmt, xb, flags=flags, sign_mask=mask, sr_seed=77, alpha=alpha)
            od = oracle.dequantize(fmt, oc, osc, oa, rows, cols)
            codes = torch.full((oc.size + 64,), 0xA5, dtype=torch.uint8, device="cuda")
            scales = torch.full((osc.size + 64,), 0xA5, dtype=torch.uint8, device="cuda")
            out, a = B.abs_quantize_dequantize(fmt, to_dev(xb), codes=codes, scales=scales, tensor_scale=ts,
                                               opts=B.make_opts(flags, mask, 77))
            out2, a2 = B.abs_quantize_dequantize(fmt, to_dev(xb), tensor_scale=ts.clone() if ts is not None else None,
                                                 opts=B.make_opts(flags, mask, 77))
            torch.cuda.synchronize()
            assert np.float32(a.item()).view(np.uint32) == np.float32(oa).view(np.uint32)
            assert np.float32(a2.item()).view(np.uint32) == np.float32(oa).view(np.uint32)
            assert_same("fused out", out.view(torch.int16).cpu().numpy().view(np.uint16), od)
            assert_same("fused out, no codes", out2.view(torch.int16).cpu().numpy().view(np.uint16), od)
            assert_same("fused codes", codes.cpu().numpy()[:oc.size].reshape(oc.shape), oc)
            assert_same("fused scales", scales.cpu().numpy()[:osc.size].reshape(osc.shape), osc)
            assert bool((codes[oc.size:] == 0xA5).all()) and bool((scales[osc.size:] == 0xA5).all())
    # groups down the columns (Sec. 4.1, weight-gradient operands): the output keeps the input's orientation
    C_ = B.ABS_F_GROUPS_DOWN_COLUMNS
    for flags in (0, H, H | S | S17, G):
        for name, rows, cols in (("cfg2", 304, 1024), ("cfg4", 64, 2064), ("cfg5", 2048, 272), ("cfg1", 16, 16)):
            xb = I.generate(name, rows, cols)
            alpha = 0.004 if flags & G else None
            ts = torch.tensor([alpha], dtype=torch.float32, device="cuda") if alpha is not None else None
            oc, osc, oa = oracle.quantize(fmt, np.ascontiguousarray(xb.T), flags=flags, sign_mask=mask, sr_seed=77,
                                          alpha=alpha, threads=THREADS)
            od = np.ascontiguousarray(oracle.dequantize(fmt, oc, osc, oa, cols, rows, threads=THREADS).T)
            codes = torch.full((oc.size + 64,), 0xA5, dtype=torch.uint8, device="cuda")
            scales = torch.full((osc.size + 64,), 0xA5, dtype=torch.uint8, device="cuda")
            out, a = B.abs_quantize_dequantize(fmt, to_dev(xb), codes=codes, scales=scales, tensor_scale=ts,
                                               opts=B.make_opts(flags | C_, mask, 77))
            out2, a2 = B.abs_quantize_dequantize(fmt, to_dev(xb), tensor_scale=ts.clone() if ts is not None else None,
                                                 opts=B.make_opts(flags | C_, mask, 77))
            torch.cuda.synchronize()
            assert np.float32(a.item()).view(np.uint32) == np.float32(oa).view(np.uint32)
            assert_same("column emulation out", out.view(torch.int16).cpu().numpy().view(np.uint16), od)
            assert_same("column emulation out, no codes", out2.view(torch.int16).cpu().numpy().view(np.uint16), od)
            assert_same("column emulation codes", codes.cpu().numpy()[:oc.size].reshape(oc.shape), oc)
            assert_same("column emulation scales", scales.cpu().numpy()[:osc.size].reshape(osc.shape), osc)
            assert bool((codes[oc.size:] == 0xA5).all()) and bool((scales[osc.size:] == 0xA5).all())
    # argument checks: other formats, unknown flags, one of the two optional outputs alone
    import ctypes
    L = B.lib()
    x = to_dev(I.generate("cfg1", 16, 64))
    out = torch.empty_like(x)
    ts = torch.zeros(1, dtype=torch.float32, device="cuda")
    buf = torch.empty(1024, dtype=torch.uint8, device="cuda")
    hopt = B.make_opts(B.ABS_F_HADAMARD16)
    assert L.abs_quantize_dequantize(3, x.data_ptr(), 16, 64, out.data_ptr(), None, None, ts.data_ptr(),
                                     ctypes.byref(hopt), None) == 5         # options exist for the 4-bit formats only
    import ctypes
    bad = B.make_opts(B.ABS_F_SCALES_SWIZZLED)
    assert L.abs_quantize_dequantize(fmt, x.data_ptr(), 16, 64, out.data_ptr(), None, None, ts.data_ptr(),
                                     ctypes.byref(bad), None) == 5
    assert L.abs_quantize_dequantize(fmt, x.data_ptr(), 16, 64, out.data_ptr(), buf.data_ptr(), None, ts.data_ptr(),
                                     None, None) == 1
    col = B.make_opts(B.ABS_F_GROUPS_DOWN_COLUMNS)
    assert L.abs_quantize_dequantize(fmt, x.data_ptr(), 8, 64, out.data_ptr(), None, None, ts.data_ptr(),
                                     ctypes.byref(col), None) == 2          # rows must be a multiple of 16
    assert L.abs_quantize_ex(fmt, x.data_ptr(), 16, 64, buf.data_ptr(), buf.data_ptr(), ts.data_ptr(),
                             ctypes.byref(col), None) == 5                  # the flag belongs to the emulation call only
    torch.cuda.synchronize()


@pytest.mark.parametrize("fmt", [2, 3, 4, 5, 6, 7])
def test_fused_quantize_dequantize_other_formats(B, oracle, fmt):
    """The emulation pass of IF3, IF6 and the block-size-8 formats (round-to-nearest, optional 17/16 factor and
    given alpha) against the oracle's quantize followed by its dequantize."""
    S17, G = B.ABS_F_SR_SCALE_17_16, B.ABS_F_ALPHA_GIVEN
    for flags in (0, S17, G):
        for name, rows, cols in (("cfg5", 300, 1024), ("cfg2", 64, 2064), ("cfg1", 1, 16)):
            xb = I.generate(name, rows, cols)
            alpha = 0.004 if flags & G else None
            ts = torch.tensor([alpha], dtype=torch.float32, device="cuda") if alpha is not None else None
            oc, osc, oa = oracle.quantize(fmt, xb, flags=flags, alpha=alpha)
            od = oracle.dequantize(fmt, oc, osc, oa, rows, cols)
            codes = torch.full((oc.size + 64,), 0xA5, dtype=torch.uint8, device="cuda")
            scales = torch.full((osc.size + 64,), 0xA5, dtype=torch.uint8, device="cuda")
            out, a = B.abs_quantize_dequantize(fmt, to_dev(xb), codes=codes, scales=scales, tensor_scale=ts,
                                               opts=B.make_opts(flags))
            out2, a2 = B.abs_quantize_dequantize(fmt, to_dev(xb), tensor_scale=ts.clone() if ts is not None else None,
                                                 opts=B.make_opts(flags))
            torch.cuda.synchronize()
            assert np.float32(a.item()).view(np.uint32) == np.float32(oa).view(np.uint32)
            assert np.float32(a2.item()).view(np.uint32) == np.float32(oa).view(np.uint32)
            assert_same("fused out", out.view(torch.int16).cpu().numpy().view(np.uint16), od)
            assert_same("fused out, no codes", out2.view(torch.int16).cpu().numpy().view(np.uint16), od)
            assert_same("fused codes", codes.cpu().numpy()[:oc.size].reshape(oc.shape), oc)
            assert_same("fused scales", scales.cpu().numpy()[:osc.size].reshape(osc.shape), osc)
            assert bool((codes[oc.size:] == 0xA5).all()) and bool((scales[osc.size:] == 0xA5).all())


@pytest.mark.parametrize("fmt", [0, 1])
def test_linear_layer_recipe(B, oracle, fmt):
    """Sec. 4.1: forward, dgrad and wgrad of an emulated quantized linear layer.  The operands the layer feeds to
    its GEMMs are rebuilt with the oracle (which dimension, which options, which seeds), the products in float64;
    the bf16 GEMM results must agree to bf16 accuracy, and the Hadamard transform must cancel in wgrad."""
    from paper_2603_28765_b200 import linear
    T, din, dout = 256, 192, 160
    rng = np.random.default_rng(3)
    xb = I.f32_to_bf16_bits(rng.standard_normal((T, din)).astype(np.float32))
    wb = I.f32_to_bf16_bits((rng.standard_normal((dout, din)) * 0.05).astype(np.float32))
    gb = I.f32_to_bf16_bits((rng.standard_normal((T, dout)) * 1e-3).astype(np.float32))
    x, w, dy = to_dev(xb), to_dev(wb), to_dev(gb)
    mask, seed = 0x5A3C, 11
    H, S, S17 = oracle.F_HADAMARD16, oracle.F_STOCHASTIC, oracle.F_SR_SCALE_17_16

    def oq(bits, flags=0, columns=False, sr_seed=0):
        src = np.ascontiguousarray(bits.T) if columns else bits
        c, s, a = oracle.quantize(fmt, src, flags=flags, sign_mask=mask, sr_seed=sr_seed)
        d = I.bf16_bits_to_f32(oracle.dequantize(fmt, c, s, a, *src.shape)).astype(np.float64)
        return d.T if columns else d

    def close(got, want):
        got = got.float().cpu().numpy().astype(np.float64)
        scale = np.abs(want).max()
        assert np.abs(got - want).max() <= 2.0 ** -7 * scale, np.abs(got - want).max() / scale

    y = linear.forward(x, w, fmt)
    close(y, oq(xb) @ oq(wb).T)
    dx, dw = linear.backward(x, w, dy, fmt, sign_mask=mask, seed=seed)
    close(dx, oq(gb, S | S17, sr_seed=seed) @ oq(wb, columns=True))
    gq, xq = oq(gb, H | S | S17, columns=True, sr_seed=seed + 1), oq(xb, H, columns=True)
    close(dw, gq.T @ xq)
    # the transform cancels: the emulated wgrad approximates dY^T X of the untransformed tensors
    exact = I.bf16_bits_to_f32(gb).astype(np.float64).T @ I.bf16_bits_to_f32(xb).astype(np.float64)
    rel = np.linalg.norm(dw.float().cpu().numpy() - exact) / np.linalg.norm(exact)
    assert rel < 0.25, rel


@pytest.mark.parametrize("fmt", [0, 1])
def test_swizzled_scale_layout(B, oracle, fmt):
    """ABS_F_SCALES_SWIZZLED: same codes and alpha, scale bytes permuted into the 128x4-tile layout (the
    oracle builds that layout by reshapes from the row-major scales); padding bytes stay untouched; the
    dequantize option reads the same layout back."""
    for name, rows, cols in (("cfg2", 300, 4096), ("cfg5", 129, 208), ("cfg1", 256, 1024)):
        xb = I.generate(name, rows, cols)
        oc, osc, oa = oracle.quantize(fmt, xb, threads=THREADS)
        x = to_dev(xb)
        nsw = B.abs_scales_bytes_swizzled(fmt, rows, cols)
        assert nsw == -(-rows // 128) * -(-(cols // 16) // 4) * 512
        scales = torch.full((nsw,), 0xEE, dtype=torch.uint8, device="cuda")
        opts = B.make_opts(B.ABS_F_SCALES_SWIZZLED)
        codes, scales, ts = B.abs_quantize(fmt, x, scales=scales, opts=opts)
        torch.cuda.synchronize()
        assert np.float32(ts.item()).view(np.uint32) == np.float32(oa).view(np.uint32)
        assert_same("codes", codes.cpu().numpy().reshape(rows, -1), oc)
        assert_same("swizzled scales", scales.cpu().numpy(), oracle.swizzle_scales(osc, fill=0xEE))
        out = B.abs_dequantize(fmt, codes, scales, ts, rows, cols, opts=opts)
        assert_same("dequant", out.view(torch.int16).cpu().numpy().view(np.uint16),
                    oracle.dequantize(fmt, oc, osc, oa, rows, cols, threads=THREADS))
    L = B.lib()
    import ctypes
    bad = B.make_opts(B.ABS_F_SCALES_SWIZZLED)
    assert L.abs_quantize_ex(2, x.data_ptr(), rows, cols, codes.data_ptr(), scales.data_ptr(), ts.data_ptr(),
                             ctypes.byref(bad), None) == 5          # IF3 has no tensor-core layout
    assert B.abs_scales_bytes_swizzled(2, 128, 64) == 0


def test_split_dequantize_and_mac_matmul(B, oracle):
    """Sec. 5.2 on the GPU.  (1) The two halves of the split dequantize are byte-identical to the oracle's.
    (2) matmul_mac (four exact-product BF16 GEMMs + FP32 factors 1, 6/7, 36/49) agrees with the float64 MAC
    reference to FP32-accumulation accuracy.  (3) The paper's own emulation (dequantize to BF16, one GEMM)
    is the same product up to the BF16 rounding of the operands -- visibly less accurate, as expected.
    Tolerances: a K-term FP32 sum carries about sqrt(K) * 2^-24 relative error on the scale of the result;
    BF16 operands carry 2^-9 per element, i.e. about 2^-9 / sqrt(K) .. 2^-9 on the result."""
    from paper_2603_28765_b200 import gemm
    m, n, k = 192, 160, 1024
    a = I.generate("cfg2", m, k)
    b = I.generate("cfg3a", n, k, seed=9)
    qa_o, qb_o = oracle.quantize(1, a, threads=THREADS), oracle.quantize(1, b, threads=THREADS)
    qa = B.abs_quantize(1, to_dev(a))
    qb = B.abs_quantize(1, to_dev(b))
    for flag, sel in ((B.ABS_F_FP_GROUPS_ONLY, oracle.F_FP_GROUPS_ONLY), (B.ABS_F_INT_GROUPS_RAW, oracle.F_INT_GROUPS_RAW)):
        got = B.abs_dequantize(1, qa[0], qa[1], qa[2], m, k, opts=B.make_opts(flag))
        want = oracle.dequantize(1, qa_o[0], qa_o[1], qa_o[2], m, k, select=sel, threads=THREADS)
        assert_same("split half", got.view(torch.int16).cpu().numpy().view(np.uint16), want)
    ref = oracle.mac_matmul_reference(1, qa_o, qb_o, m, n, k)
    scale = np.abs(ref).max()
    c_mac = gemm.matmul_mac(qa, qb, m, n, k).double().cpu().numpy()
    c_emu = gemm.matmul_emulated(qa, qb, m, n, k).double().cpu().numpy()
    err_mac = np.abs(c_mac - ref).max() / scale
    err_emu = np.abs(c_emu - ref).max() / scale
    assert err_mac < 2e-5, err_mac
    assert err_emu < 4e-3, err_emu
    assert err_mac < 0.1 * err_emu, (err_mac, err_emu)
    import ctypes
    both = B.make_opts(B.ABS_F_FP_GROUPS_ONLY | B.ABS_F_INT_GROUPS_RAW)
    out = torch.empty((m, k), dtype=torch.bfloat16, device="cuda")
    L = B.lib()
    assert L.abs_dequantize_ex(1, qa[0].data_ptr(), qa[1].data_ptr(), qa[2].data_ptr(), m, k, out.data_ptr(),
                               ctypes.byref(both), None) == 5
    one = B.make_opts(B.ABS_F_FP_GROUPS_ONLY)
    assert L.abs_dequantize_ex(0, qa[0].data_ptr(), qa[1].data_ptr(), qa[2].data_ptr(), m, k, out.data_ptr(),
                               ctypes.byref(one), None) == 5


# ------------------------------------------------------------------ dequantize of bytes no quantizer produced

def nan_aware_same(name, got, want, as_float):
    got, want = np.asarray(got), np.asarray(want)
    gn, wn = np.isnan(as_float(got)), np.isnan(as_float(want))
    assert np.array_equal(gn, wn), f"{name}: NaN positions differ ({int(gn.sum())} vs {int(wn.sum())})"
    assert_same(name, np.where(gn, 0, got), np.where(wn, 0, want))


@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_dequantize_arbitrary_bytes(B, oracle, fmt):
    """abs_dequantize on arbitrary code and scale bytes -- every scale byte 0x00..0xFF (0x7F / 0xFF: E4M3 NaN, which
    must propagate; 0x80; bit 7 set on plain NVFP4 scales), the most negative integer code, the FP code 'minus
    zero' -- against the oracle by bit pattern, bf16 and fp32 outputs, NaNs compared as 'is NaN'."""
    rows, cols = 16, 1024
    for seed, alpha in ((0, 0.0173), (1, 1.0), (2, 3.0e-20)):
        codes, scales = I.arbitrary_quantized_bytes(B.FMT_BITS[fmt], B.FMT_GROUP[fmt], rows, cols, seed)
        dc, ds = torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda()
        ts = torch.tensor([alpha], dtype=torch.float32, device="cuda")
        a32 = np.float32(ts.item())
        got16 = B.abs_dequantize(fmt, dc, ds, ts, rows, cols).view(torch.int16).cpu().numpy().view(np.uint16)
        got32 = B.abs_dequantize(fmt, dc, ds, ts, rows, cols, opts=B.make_opts(B.ABS_F_OUT_FP32)).cpu().numpy()
        want16 = oracle.dequantize(fmt, codes, scales, a32, rows, cols)
        want32 = oracle.dequantize(fmt, codes, scales, a32, rows, cols, out_fp32=True)
        assert np.isnan(want32).any()
        nan_aware_same("bf16", got16, want16, I.bf16_bits_to_f32)
        nan_aware_same("fp32", got32.view(np.uint32), want32.view(np.uint32), lambda u: u.view(np.float32))
        if fmt == 1:      # the split halves used for the MAC arithmetic read the same bytes
            for flag, sel in ((B.ABS_F_FP_GROUPS_ONLY, oracle.F_FP_GROUPS_ONLY), (B.ABS_F_INT_GROUPS_RAW, oracle.F_INT_GROUPS_RAW)):
                g = B.abs_dequantize(fmt, dc, ds, ts, rows, cols, opts=B.make_opts(flag))
                w = oracle.dequantize(fmt, codes, scales, a32, rows, cols, select=sel)
                nan_aware_same("split", g.view(torch.int16).cpu().numpy().view(np.uint16), w, I.bf16_bits_to_f32)
        if fmt in (0, 1):  # the tiled scale layout reads the same bytes from other places
            sw = torch.from_numpy(oracle.swizzle_scales(scales)).cuda()
            g = B.abs_dequantize(fmt, dc, sw, ts, rows, cols, opts=B.make_opts(B.ABS_F_SCALES_SWIZZLED))
            nan_aware_same("swizzled", g.view(torch.int16).cpu().numpy().view(np.uint16), want16, I.bf16_bits_to_f32)


def test_tensor_maximum_below_the_supported_range(B, oracle):
    """The supported range is a tensor maximum of 0 or at least 2^-100 (both sides of that line with parity are in
    the edge-tensor cases).  Below it the reciprocals of Eq. 2 can overflow: the call still succeeds, alpha is
    still Eq. 1 exactly, and the outputs are unspecified -- nothing else is promised, and nothing else is checked."""
    xb = I.below_range_tensor()
    for fmt in ALL_FMTS:
        c, s, a, _ = gpu_quantize(B, fmt, xb)
        want = oracle.alpha_from_amax(fmt, oracle.amax(xb))
        assert np.float32(a).view(np.uint32) == np.float32(want).view(np.uint32)
    torch.cuda.synchronize()


# ------------------------------------------------------------------ row shards through the product calls

@pytest.mark.parametrize("fmt", [0, 1, 2, 3, 6])
@pytest.mark.parametrize("opt", ["rtn", "sr", "hsr17"])
def test_row_shards_through_the_library_equal_one_call(B, oracle, fmt, opt):
    """The multi-GPU protocol with the library's own calls, run on one GPU: every shard reduces its rows with
    abs_amax, the maxima are combined on the host (the one 4-byte exchange), every shard is quantized with
    abs_quantize_ex(ABS_F_ALPHA_GIVEN) and, for stochastic rounding, the index of its first element as
    sr_index_offset.  Codes and scales concatenated must equal one abs_quantize_ex call on the whole tensor and
    the oracle, byte for byte; so must alpha."""
    flags = {"rtn": 0, "sr": B.ABS_F_STOCHASTIC,
             "hsr17": B.ABS_F_HADAMARD16 | B.ABS_F_STOCHASTIC | B.ABS_F_SR_SCALE_17_16}[opt]
    mask, seed = oracle.hadamard_sign_mask(3), 0x1234567890ABCDEF
    xb = I.generate("cfg4" if flags else "cfg2", 600, 2048)
    rows, cols = xb.shape
    whole_c, whole_s, whole_a, _ = gpu_quantize(B, fmt, xb, flags, mask, seed)
    oc, osc, oa = oracle.quantize(fmt, xb, flags=flags, sign_mask=mask, sr_seed=seed, threads=THREADS)
    assert np.float32(whole_a).view(np.uint32) == np.float32(oa).view(np.uint32)
    assert_same("whole codes", whole_c, oc)
    assert_same("whole scales", whole_s, osc)
    bounds = [(0, 256), (256, 257), (257, 600)]
    shards = [to_dev(np.ascontiguousarray(xb[lo:hi])) for lo, hi in bounds]
    amax_opts = B.make_opts(flags & B.ABS_F_HADAMARD16, mask)
    local_max = [float(B.abs_amax(x, opts=amax_opts).item()) for x in shards]
    alpha = B.abs_alpha_from_amax(fmt, max(local_max))                  # host max = the all-reduce(max) of 4 bytes
    assert np.float32(alpha).view(np.uint32) == np.float32(oa).view(np.uint32)
    cs, ss = [], []
    for (lo, hi), x in zip(bounds, shards):
        ts = torch.tensor([alpha], dtype=torch.float32, device="cuda")
        o = B.make_opts(flags | B.ABS_F_ALPHA_GIVEN, mask, seed, lo * cols)
        c, s, _ = B.abs_quantize(fmt, x, tensor_scale=ts, opts=o)
        cs.append(c.cpu().numpy().reshape(hi - lo, -1))
        ss.append(s.cpu().numpy().reshape(hi - lo, -1))
    assert_same("shard codes", np.concatenate(cs), oc)
    assert_same("shard scales", np.concatenate(ss), osc)
    if flags & B.ABS_F_STOCHASTIC:
        import ctypes
        L = B.lib()
        bad = B.make_opts(flags | B.ABS_F_ALPHA_GIVEN, mask, seed, 8)           # not a multiple of 16
        x = shards[0]
        ts = torch.tensor([alpha], dtype=torch.float32, device="cuda")
        assert L.abs_quantize_ex(fmt, x.data_ptr(), 256, cols, c.data_ptr(), s.data_ptr(), ts.data_ptr(),
                                 ctypes.byref(bad), None) == 2


@pytest.mark.parametrize("fmt", [0, 1])
def test_index_offset_in_the_other_stochastic_entry_points(B, oracle, fmt):
    """sr_index_offset in abs_quantize_dequantize (both orientations) and abs_quantize_transposed: a matrix quantized
    on its own with the offset of its first element equals the corresponding rows of the larger tensor."""
    flags = B.ABS_F_STOCHASTIC | B.ABS_F_SR_SCALE_17_16
    seed = 4242
    xb = I.generate("cfg4", 96, 512)
    oc, osc, oa = oracle.quantize(fmt, xb, flags=flags, sr_seed=seed)
    od = oracle.dequantize(fmt, oc, osc, oa, 96, 512)
    lo = 32
    part = np.ascontiguousarray(xb[lo:])
    ts = torch.tensor([float(oa)], dtype=torch.float32, device="cuda")
    out, _ = B.abs_quantize_dequantize(fmt, to_dev(part), tensor_scale=ts,
                                       opts=B.make_opts(flags | B.ABS_F_ALPHA_GIVEN, 0, seed, lo * 512))
    assert_same("emulation shard", out.view(torch.int16).cpu().numpy().view(np.uint16), od[lo:])
    # transposed: the index runs over X^T [512, 96]; the last 64 columns of X are rows 448.. of X^T
    xt = np.ascontiguousarray(xb.T)
    tc, tsc, ta = oracle.quantize(fmt, xt, flags=flags, sr_seed=seed)
    cols_part = np.ascontiguousarray(xb[:, 448:])
    ts = torch.tensor([float(ta)], dtype=torch.float32, device="cuda")
    ct, st, _ = B.abs_quantize_transposed(fmt, to_dev(cols_part), tensor_scale=ts,
                                          opts=B.make_opts(flags | B.ABS_F_ALPHA_GIVEN, 0, seed, 448 * 96))
    assert_same("transposed shard codes", ct.cpu().numpy().reshape(64, -1), tc[448:])
    assert_same("transposed shard scales", st.cpu().numpy().reshape(64, -1), tsc[448:])


def test_tensor_core_consumer_reads_codes_and_swizzled_scales(B, oracle):
    """Sec. 3: a group stored as FP4 is an NVFP4 group, so a plain-NVFP4 tensor from this library -- packed codes,
    E4M3 scales in the 128x4-tile layout (ABS_F_SCALES_SWIZZLED), FP32 tensor scale -- must be directly usable as an
    operand of Blackwell's block-scaled FP4 tensor-core product.  The consumer here is the block-scaled matrix
    product that PyTorch exposes (a library kernel, operands in this GPU's memory): it is given the library's
    buffers as they are, and its FP32 result is compared with the float64 product of the oracle's dequantized
    operands.  Every product of two codes and two scales is exact and the sums are accumulated in FP32, so the
    tolerance is that of an FP32 sum over K terms."""
    F = torch.nn.functional
    if not (hasattr(F, "scaled_mm") and hasattr(torch, "float4_e2m1fn_x2")):
        pytest.skip("this PyTorch has no block-scaled FP4 matrix product")
    for (m, n, k) in ((256, 384, 1024), (128, 128, 64), (640, 256, 4096)):
        a, b = I.generate("cfg2", m, k), I.generate("cfg3a", n, k, seed=9)
        sw = B.make_opts(B.ABS_F_SCALES_SWIZZLED)
        ca, sa, aa = B.abs_quantize(0, to_dev(a), opts=sw)
        cb, sb, ab = B.abs_quantize(0, to_dev(b), opts=sw)
        torch.cuda.synchronize()
        qa, qb = oracle.quantize(0, a, threads=THREADS), oracle.quantize(0, b, threads=THREADS)
        ref = oracle.mac_matmul_reference(0, qa, qb, m, n, k)
        a4 = ca.view(m, k // 2).view(torch.float4_e2m1fn_x2)
        b4 = cb.view(n, k // 2).view(torch.float4_e2m1fn_x2)
        block, tensor = F.ScalingType.BlockWise1x16, F.ScalingType.TensorWise
        tiled, plain = F.SwizzleType.SWIZZLE_32_4_4, F.SwizzleType.NO_SWIZZLE
        c = F.scaled_mm(a4, b4.t(), scale_a=[sa.view(torch.float8_e4m3fn), aa], scale_recipe_a=[block, tensor],
                        scale_b=[sb.view(torch.float8_e4m3fn), ab], scale_recipe_b=[block, tensor],
                        swizzle_a=[tiled, plain], swizzle_b=[tiled, plain], output_dtype=torch.float32)
        torch.cuda.synchronize()
        err = np.abs(c.double().cpu().numpy() - ref).max() / np.abs(ref).max()
        assert err < 2e-6, (m, n, k, err)


@pytest.mark.parametrize("fmt", [0, 1])
def test_tensor_core_matmul_matches_mac_reference(B, oracle, fmt):
    """abs_matmul (hand-written tcgen05 kernel: TMA-fed block-scaled FP4 MMAs, three accumulators for the FP x FP,
    mixed and INT x INT group pairs, factors 1, 6/7, 36/49 in the FP32 epilogue) against the float64 reference of the
    MAC arithmetic of Sec. 5.2.  Every code product is exact; the difference is the FP32 accumulation of the tensor
    core over K terms, so the tolerance is that of an FP32 sum (2e-5 of the largest |C| is ample up to K = 4096)."""
    for (m, n, k) in ((128, 128, 256), (256, 384, 1024), (128, 256, 4096), (640, 128, 512), (1, 128, 256), (100, 256, 512), (333, 128, 1024)):
        a, b = I.generate("cfg2", m, k), I.generate("cfg3a", n, k, seed=9)
        qa, qb = B.abs_quantize(fmt, to_dev(a)), B.abs_quantize(fmt, to_dev(b))
        oa, ob = oracle.quantize(fmt, a, threads=THREADS), oracle.quantize(fmt, b, threads=THREADS)
        ref = oracle.mac_matmul_reference(fmt, oa, ob, m, n, k)
        c = B.abs_matmul(fmt, qa, qb, m, n, k, check=True).double().cpu().numpy()
        err = np.abs(c - ref).max() / np.abs(ref).max()
        assert err < 2e-5, (fmt, m, n, k, err)
        if fmt == 1:
            assert 0.05 < float((oa[1] >> 7).mean()) < 0.95     # both kinds of groups take part
    # a partial last row block: nothing is written below row m
    m, n, k = 100, 128, 256
    qa, qb = B.abs_quantize(fmt, to_dev(I.generate("cfg2", m, k))), B.abs_quantize(fmt, to_dev(I.generate("cfg3a", n, k, seed=9)))
    guard = torch.full((128, n), 7.0, dtype=torch.float32, device="cuda")
    B.abs_matmul(fmt, qa, qb, m, n, k, out=guard, check=True)
    assert bool((guard[m:] == 7.0).all()) and not bool((guard[:m] == 7.0).all())
    # shapes the kernel does not take, and other formats
    L = B.lib()
    assert L.abs_matmul_workspace_bytes(fmt, 128, 100, 256) == 0 and L.abs_matmul_workspace_bytes(fmt, 128, 128, 128) == 0
    assert L.abs_matmul_workspace_bytes(2, 128, 128, 256) == 0
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    out = torch.empty((128, 128), dtype=torch.float32, device="cuda")
    args = (qa[0].data_ptr(), qa[1].data_ptr(), qa[2].data_ptr(), qb[0].data_ptr(), qb[1].data_ptr(), qb[2].data_ptr())
    assert L.abs_matmul(fmt, *args, 128, 128, 192, out.data_ptr(), ws.data_ptr(), 4096, None) == 2      # k % 256
    assert L.abs_matmul(3, *args, 128, 128, 256, out.data_ptr(), ws.data_ptr(), 4096, None) == 4        # format
    assert L.abs_matmul(fmt, *args, 128, 128, 256, out.data_ptr(), ws.data_ptr(), 4096, None) in (3, 7)  # alignment or size


def test_calls_without_scratch_replay_from_a_cuda_graph(B, oracle):
    """The header allows capturing the calls that use no scratch: abs_quantize_ex with ABS_F_ALPHA_GIVEN and
    abs_dequantize.  Captured once, replayed on two different tensors copied into the same input buffer, the
    outputs must be the oracle's both times."""
    rows, cols = 96, 1024
    xs = [I.generate("cfg1", rows, cols, seed=s) for s in (3, 4)]
    alpha = 0.0042
    x = torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda")
    ts = torch.tensor([alpha], dtype=torch.float32, device="cuda")
    codes = torch.empty(rows * cols // 2, dtype=torch.uint8, device="cuda")
    scales = torch.empty(rows * cols // 16, dtype=torch.uint8, device="cuda")
    out = torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda")
    opts = B.make_opts(B.ABS_F_ALPHA_GIVEN)
    B.abs_quantize(1, x, codes, scales, ts, opts=opts)            # first call on the device happens outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            B.abs_quantize(1, x, codes, scales, ts, opts=opts, stream=s)
            B.abs_dequantize(1, codes, scales, ts, rows, cols, out=out, stream=s)
    for xb in xs:
        x.copy_(to_dev(xb))
        g.replay()
        torch.cuda.synchronize()
        oc, osc, oa = oracle.quantize(1, xb, flags=oracle.F_ALPHA_GIVEN, alpha=alpha)
        assert_same("graph codes", codes.cpu().numpy().reshape(rows, -1), oc)
        assert_same("graph scales", scales.cpu().numpy().reshape(rows, -1), osc)
        assert_same("graph dequant", out.view(torch.int16).cpu().numpy().view(np.uint16),
                    oracle.dequantize(1, oc, osc, oa, rows, cols))


@pytest.mark.parametrize("fmt", [0, 1])
def test_tensor_core_matmul_on_arbitrary_bytes(B, oracle, fmt):
    """abs_matmul on operands that no quantizer produced: random code bytes (every nibble, the most negative integer
    code and FP minus zero included) and random finite scale bytes with and without bit 7 -- all-FP tensors, all-integer
    tensors and mixtures, so each of the three accumulators is exercised alone and together -- against the float64
    reference built from the oracle's dequantize.  Plain NVFP4 must ignore bit 7 of its scale bytes."""
    m, n, k = 128, 256, 512
    rng = np.random.default_rng(5)
    for a_flags, b_flags in (("mixed", "mixed"), ("fp", "fp"), ("int", "int"), ("fp", "int"), ("int", "mixed")):
        ops = []
        for rows, kind in ((m, a_flags), (n, b_flags)):
            codes = rng.integers(0, 256, (rows, k // 2), dtype=np.uint8)
            mag = rng.integers(0x20, 0x50, (rows, k // 16), dtype=np.uint8)       # scales 2^-3 .. 2^3: sums stay moderate
            bit7 = {"fp": 0, "int": 0x80}.get(kind)
            if bit7 is None:
                bit7 = (rng.integers(0, 2, mag.shape, dtype=np.uint8) << 7).astype(np.uint8)
            scales = (mag | bit7).astype(np.uint8)
            scales[rows // 2, :4] = [0x00, 0x80, 0x01, 0x7E]                       # zero scale, flagged zero, smallest, largest
            ops.append((codes, scales, np.float32(0.75 if rows == m else 1.5)))
        ref = oracle.mac_matmul_reference(fmt, ops[0], ops[1], m, n, k)
        dev = [(torch.from_numpy(c).cuda(), torch.from_numpy(s).cuda(), torch.tensor([a], dtype=torch.float32, device="cuda"))
               for c, s, a in ops]
        c = B.abs_matmul(fmt, dev[0], dev[1], m, n, k, check=True).double().cpu().numpy()
        err = np.abs(c - ref).max() / np.abs(ref).max()
        assert err < 2e-5, (fmt, a_flags, b_flags, err)


def test_scratch_ring_overrun_is_reported(B, oracle):
    """More than ABS_MAX_INFLIGHT amax-carrying calls enqueued between the two kernels of one call: that call loses
    its maximum.  Provoked without any fault: stream A first runs a bounded delay kernel, then one abs_quantize;
    while A is delayed, stream B runs 1100 abs_quantize calls, which wraps the ring of 1024 slots past A's slot.
    A's group-quantize kernel then finds another call's tag in its slot and raises the flag: the next call that
    takes a slot returns ABS_ERR_SIZE (7) exactly once, and the library works normally afterwards."""
    import ctypes
    L = B.lib()
    xb = I.generate("cfg1", 64, 256)
    x = to_dev(xb)
    a, b = torch.cuda.Stream(), torch.cuda.Stream()
    outs_b = B.abs_quantize(1, x)                      # buffers reused by every call on stream B
    codes_a, scales_a, ts_a = B.abs_quantize(1, x)
    torch.cuda.synchronize()
    with torch.cuda.stream(a):
        torch.cuda._sleep(400_000_000)                  # about 0.2 s at 2 GHz: a bounded busy-wait, nothing else
        B.abs_quantize(1, x, codes_a, scales_a, ts_a, stream=a)
    for _ in range(1100):
        B.abs_quantize(1, x, outs_b[0], outs_b[1], outs_b[2], stream=b)
    torch.cuda.synchronize()
    sp = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    args = (1, x.data_ptr(), 64, 256, outs_b[0].data_ptr(), outs_b[1].data_ptr(), outs_b[2].data_ptr(), sp)
    assert L.abs_quantize(*args) == 7                   # the overrun of the delayed call is reported here ...
    assert L.abs_quantize(*args) == 0                   # ... once
    torch.cuda.synchronize()
    assert float(ts_a.item()) == 1.0                    # the overrun call fell back to alpha = 1, visibly
    check_case(B, oracle, 1, xb)                        # and everything is back to normal


@pytest.mark.parametrize("fmt,m,n,k", [(1, 4096, 4096, 4096), (0, 4096, 4096, 4096), (1, 1920, 2176, 1024), (0, 1920, 2176, 1024)])
def test_tensor_core_matmul_full_size_sampled(B, oracle, fmt, m, n, k):
    """abs_matmul at 4096 x 4096 x 4096 (the size its timing is quoted on) and at a size whose tile rows do not fill
    the last band of the tile walk: every block of the persistent kernel computes several tiles here.  48 sampled rows
    of A against 48 sampled rows of B give a 48 x 48 sample of C, spread over the tiles, that the float64 reference
    can compute; first and last rows included."""
    a, b = I.generate("cfg2", m, k), I.generate("cfg3a", n, k, seed=9)
    qa, qb = B.abs_quantize(fmt, to_dev(a)), B.abs_quantize(fmt, to_dev(b))
    c = B.abs_matmul(fmt, qa, qb, m, n, k, check=True)
    rng = np.random.default_rng(17)
    ra = np.array(sorted(set([0, m - 1] + [int(v) for v in rng.integers(0, m, 46)])))
    rb = np.array(sorted(set([0, n - 1] + [int(v) for v in rng.integers(0, n, 46)])))
    alpha_a, alpha_b = np.float32(qa[2].item()), np.float32(qb[2].item())
    oa = oracle.quantize(fmt, np.ascontiguousarray(a[ra]), flags=oracle.F_ALPHA_GIVEN, alpha=alpha_a)
    ob = oracle.quantize(fmt, np.ascontiguousarray(b[rb]), flags=oracle.F_ALPHA_GIVEN, alpha=alpha_b)
    assert np.array_equal(qa[0].view(m, k // 2)[torch.from_numpy(ra).cuda()].cpu().numpy(), oa[0])     # same operands
    ref = oracle.mac_matmul_reference(fmt, oa, ob, len(ra), len(rb), k)
    got = c[torch.from_numpy(ra).cuda()][:, torch.from_numpy(rb).cuda()].double().cpu().numpy()
    scale = float(c.abs().max().item())
    assert np.abs(got - ref).max() <= 2e-5 * scale, np.abs(got - ref).max() / scale
    # and every tile was written by the block that owns it: the whole of C against the split path (four cuBLAS GEMMs)
    if fmt == 1:
        from paper_2603_28765_b200 import gemm
        other = gemm.matmul_mac_split(qa, qb, m, n, k).float()
        assert float((c - other).abs().max().item()) <= 2e-6 * scale


@pytest.mark.parametrize("fmt", [0, 1])
def test_weight_gradient_product_from_transposed_quantize(B, oracle, fmt):
    """Sec. 4.1: for the weight-gradient product dW = dY^T X both operands are quantized along the token dimension.
    abs_quantize_transposed writes exactly the K-major codes and scales abs_matmul reads (K = tokens), so the two
    calls compose without any layout step: dW from the library against the float64 MAC reference on the oracle's
    quantization of the transposed operands."""
    tokens, d_out, d_in = 512, 256, 128
    rng = np.random.default_rng(23)
    dy = I.f32_to_bf16_bits((rng.standard_normal((tokens, d_out)) * 1e-3).astype(np.float32))
    x = I.f32_to_bf16_bits(rng.standard_normal((tokens, d_in)).astype(np.float32))
    q_dy = B.abs_quantize_transposed(fmt, to_dev(dy))          # dY^T [d_out, tokens], groups along the tokens
    q_x = B.abs_quantize_transposed(fmt, to_dev(x))            # X^T  [d_in,  tokens]
    dw = B.abs_matmul(fmt, q_dy, q_x, d_out, d_in, tokens, check=True).double().cpu().numpy()
    o_dy = oracle.quantize(fmt, np.ascontiguousarray(dy.T), threads=THREADS)
    o_x = oracle.quantize(fmt, np.ascontiguousarray(x.T), threads=THREADS)
    ref = oracle.mac_matmul_reference(fmt, o_dy, o_x, d_out, d_in, tokens)
    assert np.abs(dw - ref).max() <= 2e-5 * np.abs(ref).max()
    exact = I.bf16_bits_to_f32(dy).astype(np.float64).T @ I.bf16_bits_to_f32(x).astype(np.float64)
    rel = np.linalg.norm(dw - exact) / np.linalg.norm(exact)
    assert rel < 0.2, rel                                        # and it is the weight gradient, up to the quantization error


def test_linear_layer_on_the_tensor_cores(B, oracle):
    """The quantized linear layer of Sec. 4.1 without the BF16 detour (linear.forward_tc / backward_tc): three
    tensor-core products of operands quantized K-major by abs_quantize / abs_quantize_transposed, the gradient
    operands with Hadamard, stochastic rounding and the 17/16 factor.  Each product is compared with the float64 MAC
    reference on the oracle's quantization of the same operand with the same options (so this also pins that the
    options and seeds reach the right operand), and with the exact product up to the quantization error."""
    from paper_2603_28765_b200 import linear
    tokens, d_in, d_out = 768, 256, 512        # each of them is the K of one product: multiples of 256
    mask, seed = 0x5A3C, 77
    rng = np.random.default_rng(31)
    x = I.f32_to_bf16_bits(rng.standard_normal((tokens, d_in)).astype(np.float32))
    w = I.f32_to_bf16_bits((rng.standard_normal((d_out, d_in)) * 0.05).astype(np.float32))
    dy = I.f32_to_bf16_bits((rng.standard_normal((tokens, d_out)) * 1e-3).astype(np.float32))
    xd, wd, dyd = to_dev(x), to_dev(w), to_dev(dy)
    T = lambda a: np.ascontiguousarray(a.T)
    SR = oracle.F_STOCHASTIC | oracle.F_SR_SCALE_17_16
    tol = lambda ref: 2e-5 * np.abs(ref).max()

    y = linear.forward_tc(xd, wd).double().cpu().numpy()
    ref = oracle.mac_matmul_reference(1, oracle.quantize(1, x, threads=THREADS), oracle.quantize(1, w, threads=THREADS),
                                      tokens, d_out, d_in)
    assert np.abs(y - ref).max() <= tol(ref)

    dx, dw = linear.backward_tc(xd, wd, dyd, sign_mask=mask, seed=seed)
    dx, dw = dx.double().cpu().numpy(), dw.double().cpu().numpy()
    ref_dx = oracle.mac_matmul_reference(1, oracle.quantize(1, dy, flags=SR, sr_seed=seed, threads=THREADS),
                                         oracle.quantize(1, T(w), threads=THREADS), tokens, d_in, d_out)
    assert np.abs(dx - ref_dx).max() <= tol(ref_dx)
    H = oracle.F_HADAMARD16
    ref_dw = oracle.mac_matmul_reference(1, oracle.quantize(1, T(dy), flags=H | SR, sign_mask=mask, sr_seed=seed + 1, threads=THREADS),
                                         oracle.quantize(1, T(x), flags=H, sign_mask=mask, threads=THREADS), d_out, d_in, tokens)
    assert np.abs(dw - ref_dw).max() <= tol(ref_dw)

    f = lambda a: I.bf16_bits_to_f32(a).astype(np.float64)
    for got, exact in ((y, f(x) @ f(w).T), (dx, f(dy) @ f(w)), (dw, f(dy).T @ f(x))):
        rel = np.linalg.norm(got - exact) / np.linalg.norm(exact)
        assert rel < 0.2, rel                       # the Hadamard transform of the two wgrad operands cancels in the product
    # and the emulated layer (BF16 GEMMs on dequantized operands) gives the same products up to its BF16 roundings
    y_e = linear.forward(xd, wd).double().cpu().numpy()
    assert np.linalg.norm(y - y_e) / np.linalg.norm(y) < 1e-2


def test_matmul_wait_limit_is_reported_and_the_next_call_works(B, oracle):
    """Every wait inside the product kernel is bounded (one second).  The self-test entry announces the loads of one
    pipeline step and never issues them: no fault and no unbounded wait, the blocks give up, set the error word, free
    their tensor memory and return; abs_matmul_check reports it, and the next ordinary call on the same workspace
    gives the right result again."""
    import time
    m, n, k = 256, 256, 1024
    a, b = I.generate("cfg2", m, k), I.generate("cfg3a", n, k, seed=9)
    qa, qb = B.abs_quantize(1, to_dev(a)), B.abs_quantize(1, to_dev(b))
    L = B.lib()
    need = L.abs_matmul_workspace_bytes(1, m, n, k)
    ws = torch.empty(need + 1024, dtype=torch.uint8, device="cuda")
    off = (-ws.data_ptr()) % 1024
    good = B.abs_matmul(1, qa, qb, m, n, k, workspace=ws, check=True).clone()
    out = torch.zeros((m, n), dtype=torch.float32, device="cuda")
    args = (1, qa[0].data_ptr(), qa[1].data_ptr(), qa[2].data_ptr(), qb[0].data_ptr(), qb[1].data_ptr(), qb[2].data_ptr(),
            m, n, k, out.data_ptr(), ws.data_ptr() + off, need, None)
    t0 = time.time()
    assert L.abs_selftest_matmul_stall(*args, 2) == 0                      # the launch itself succeeds
    assert L.abs_matmul_check(ws.data_ptr() + off, None) == 6              # ABS_ERR_CUDA: a wait ran out
    assert time.time() - t0 < 20.0
    assert L.abs_selftest_matmul_stall(*args, -1) == 2                     # not a way to make an ordinary call
    again = B.abs_matmul(1, qa, qb, m, n, k, workspace=ws, check=True)
    assert torch.equal(again, good)


@pytest.mark.parametrize("fmt", [0, 1])
def test_tensor_core_matmul_long_k_and_nan_scales(B, oracle, fmt):
    """Two corners of abs_matmul: a long contraction (K = 14336: 56 pipeline steps, the stage and slot phases wrap many
    times) against the float64 reference, and E4M3 NaN scale bytes (0x7F, and 0xFF for IF4), which must make exactly
    the rows of C that belong to their row of A, and the columns that belong to their row of B, NaN -- as dequantize
    does -- and leave every other entry equal to the reference."""
    m, n, k = 128, 128, 14336
    a, b = I.generate("cfg3a", m, k, seed=3), I.generate("cfg3a", n, k, seed=4)
    qa, qb = B.abs_quantize(fmt, to_dev(a)), B.abs_quantize(fmt, to_dev(b))
    oa, ob = oracle.quantize(fmt, a, threads=THREADS), oracle.quantize(fmt, b, threads=THREADS)
    ref = oracle.mac_matmul_reference(fmt, oa, ob, m, n, k)
    c = B.abs_matmul(fmt, qa, qb, m, n, k, check=True).double().cpu().numpy()
    assert np.abs(c - ref).max() <= 4e-5 * np.abs(ref).max()

    m, n, k = 256, 128, 512
    a, b = I.generate("cfg2", m, k), I.generate("cfg3a", n, k, seed=9)
    oa, ob = oracle.quantize(fmt, a, threads=THREADS), oracle.quantize(fmt, b, threads=THREADS)
    sa, sb = oa[1].copy(), ob[1].copy()
    sa[5, 3] = 0x7F
    sa[200, 0] = 0xFF if fmt == 1 else 0x7F
    sb[77, 31] = 0x7F
    dev = lambda q, s: (torch.from_numpy(q[0]).cuda(), torch.from_numpy(s).cuda(), torch.tensor([q[2]], dtype=torch.float32, device="cuda"))
    c = B.abs_matmul(fmt, dev(oa, sa), dev(ob, sb), m, n, k, check=True).double().cpu().numpy()
    bad = np.zeros((m, n), dtype=bool)
    bad[5, :] = bad[200, :] = True
    bad[:, 77] = True
    assert np.isnan(c[bad]).all() and np.isfinite(c[~bad]).all()
    ref = oracle.mac_matmul_reference(fmt, oa, ob, m, n, k)
    assert np.abs(c[~bad] - ref[~bad]).max() <= 2e-5 * np.abs(ref).max()
    # an all-zero operand (every scale byte zero) gives an all-zero product, not NaN
    z = np.zeros((m, k), dtype=np.uint16)
    qz = B.abs_quantize(fmt, to_dev(z))
    assert int(qz[1].max().item()) == 0
    cz = B.abs_matmul(fmt, qz, B.abs_quantize(fmt, to_dev(b)), m, n, k, check=True)
    assert bool((cz == 0).all())


@pytest.mark.parametrize("fmt", [0, 1])
def test_tensor_core_matmul_bf16_output_is_the_rounded_fp32_output(B, oracle, fmt):
    """abs_matmul_bf16 writes the FP32 result of abs_matmul rounded to nearest even: bit for bit the bf16 conversion of
    the FP32 output, on full and partial row blocks, and nothing below row m."""
    for (m, n, k) in ((256, 384, 1024), (100, 128, 256), (1152, 256, 512)):
        a, b = I.generate("cfg2", m, k), I.generate("cfg3a", n, k, seed=9)
        qa, qb = B.abs_quantize(fmt, to_dev(a)), B.abs_quantize(fmt, to_dev(b))
        c32 = B.abs_matmul(fmt, qa, qb, m, n, k, check=True)
        guard = torch.full((m + 28, n), 3.0, dtype=torch.bfloat16, device="cuda")
        B.abs_matmul(fmt, qa, qb, m, n, k, out=guard, check=True, bf16=True)
        assert torch.equal(guard[:m], c32.to(torch.bfloat16)), (fmt, m, n, k)
        assert bool((guard[m:] == 3.0).all())


@pytest.mark.parametrize("fmt", [0, 1])
def test_matmul_leaves_the_tensor_scale_of_its_output(B, oracle, fmt):
    """abs_matmul_bf16_scaled: the epilogue's running maximum of |C| gives the alpha of Eq. 1 for the next quantizer.
    It must be the very float abs_quantize computes with its own pass over C (for several next formats), on full and
    partial row blocks, so that quantizing C with ABS_F_ALPHA_GIVEN and that alpha gives the same bytes."""
    for (m, n, k) in ((256, 384, 1024), (100, 128, 256), (2048, 2048, 512)):
        a, b = I.generate("cfg2", m, k), I.generate("cfg3a", n, k, seed=9)
        qa, qb = B.abs_quantize(fmt, to_dev(a)), B.abs_quantize(fmt, to_dev(b))
        for next_fmt in (1, 2, 3):
            c, alpha = B.abs_matmul(fmt, qa, qb, m, n, k, bf16=True, next_fmt=next_fmt, check=True)
            codes, scales, alpha_own = B.abs_quantize(next_fmt, c)
            assert float(alpha.item()) == float(alpha_own.item()), (fmt, m, n, k, next_fmt)
            og = B.make_opts(B.ABS_F_ALPHA_GIVEN)
            codes2, scales2, _ = B.abs_quantize(next_fmt, c, tensor_scale=alpha.clone(), opts=og)
            assert torch.equal(codes, codes2) and torch.equal(scales, scales2)
    # an all-zero product: alpha 1, as the quantizer's own pass gives
    z = to_dev(np.zeros((128, 256), dtype=np.uint16))
    c, alpha = B.abs_matmul(fmt, B.abs_quantize(fmt, z), B.abs_quantize(fmt, to_dev(I.generate("cfg3a", 128, 256, seed=9))),
                            128, 128, 256, bf16=True, next_fmt=1, check=True)
    assert float(alpha.item()) == 1.0 and bool((c == 0).all())

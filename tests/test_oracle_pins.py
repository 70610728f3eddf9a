"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Every test here compares the oracle with something other than itself: values the paper
prints (tests/golden/*.txt, each file cites its source), the definition of the grids,
library conversions (torch's float8 / bfloat16 casts), brute force in float64 on small
inputs, algebraic identities, and statistics.
"""
import os

import numpy as np
import pytest

from paper_2603_28765_b200 import inputs as I

GOLD = os.path.join(os.path.dirname(__file__), "golden")
IF_FMTS = [1, 2, 3, 4]
ALL_FMTS = [0, 1, 2, 3, 4]


def read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split(":")
            out[k.strip()] = v.split()
    return out


def unpack_bitstream(codes_row_bytes, b):
    """Independent unpack: little-endian bitstream, code j at bits [b*j, b*j+b)."""
    bits = np.unpackbits(np.asarray(codes_row_bytes, dtype=np.uint8), bitorder="little")
    bits = bits.reshape(-1, b)
    return (bits * (1 << np.arange(b))).sum(axis=1)


def fp_grid(fmt):
    """Magnitude grids written out from the format definitions (Sec. 1; Sec. 5.1)."""
    if fmt in (0, 1):
        return [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    if fmt == 2:
        return [0, 1, 2, 4]
    if fmt == 3:  # E2M3, bias 1
        return [m / 8 for m in range(8)] + [(1 + m / 8) * 2 ** (e - 1) for e in (1, 2, 3) for m in range(8)]
    if fmt == 4:  # E3M2, bias 3
        return [m / 16 for m in range(4)] + [(1 + m / 4) * 2.0 ** (e - 3) for e in range(1, 8) for m in range(4)]
    raise KeyError(fmt)


def e4m3_grid():
    return [m * 2.0 ** -9 for m in range(8)] + [(8 + m) * 2.0 ** (e - 10) for e in range(1, 16) for m in range(8)][:119]


# --------------------------------------------------------------------------- paper-printed values

def test_worked_example_fig3a(oracle):
    g = read_golden("fig3a_worked_example.txt")
    X = [float(v) for v in g["X"]]
    x = np.zeros((1, 16), np.float32)
    x[0, :4] = X
    xb = I.f32_to_bf16_bits(x)
    # alpha = 1 reproduces the table literally (the pseudocode has no tensor scale).
    c4, s4, _, efp, eint = oracle.quantize(1, xb, flags=oracle.F_ALPHA_GIVEN, alpha=1.0, debug=True)
    cn, sn, _ = oracle.quantize(0, xb, flags=oracle.F_ALPHA_GIVEN, alpha=1.0)
    delta = float(oracle.e4m3_value(int(s4[0, 0])))
    assert delta == float(g["step2_delta_e4m3"][0]) == float(g["step1_delta"][0])
    xbar = np.array(X) / delta
    assert [f"{v:.2f}" for v in xbar] == [f"{float(v):.2f}" for v in g["step3_xbar"]]
    fp_codes = unpack_bitstream(cn[0], 4)[:4]
    fp_vals = [fp_grid(0)[c & 7] for c in fp_codes]
    assert fp_vals == [float(v) for v in g["step4_fp"]]
    d_fp = I.bf16_bits_to_f32(oracle.dequantize(0, cn, sn, 1.0, 1, 16))[0, :4]
    assert list(d_fp) == [float(v) for v in g["step5_d_fp"]]
    assert float(efp[0, 0]) == float(g["step6_e_fp"][0])
    assert s4[0, 0] >> 7 == 1, "step 10 selects the integer candidate"
    int_codes = unpack_bitstream(c4[0], 4)[:4]
    assert list(int_codes) == [int(v) for v in g["step7_int"]] == [int(v) for v in g["step10_selected"]]
    d_int = I.bf16_bits_to_f32(oracle.dequantize(1, c4, s4, 1.0, 1, 16))[0, :4]
    assert list(d_int) == [float(v) for v in g["step8_d_int"]]
    assert float(eint[0, 0]) == float(g["step9_e_int"][0])
    # The full path (Eq. 1 included): alpha = 42 / 2688 = 2^-6, scale saturates at 448, flag set.
    c, s, a = oracle.quantize(1, xb)
    assert a == np.float32(2.0 ** -6) and s[0, 0] == 0xFE
    assert c[0].tobytes() == bytes([0x31, 0x76, 0, 0, 0, 0, 0, 0])
    assert list(I.bf16_bits_to_f32(oracle.dequantize(1, c, s, a, 1, 16))[0, :4]) == X


def test_table1_mse_normal(oracle):
    g = read_golden("table1_mse.txt")
    xb = I.generate("cfg1", 1024, 1024)
    xf = I.bf16_bits_to_f32(xb).astype(np.float64)
    for name, fmt in (("NVFP4", 0), ("IF4", 1)):
        c, s, a = oracle.quantize(fmt, xb, threads=4)
        d = oracle.dequantize(fmt, c, s, a, 1024, 1024, out_fp32=True, threads=4).astype(np.float64)
        mse = np.mean((d - xf) ** 2) * 1e3
        assert abs(mse - float(g[name][0])) < 0.1, (name, mse)
    # the per-group error sums of the two candidates (steps 5-6 and 8-9 of Fig. 3a), before selection: the FP
    # candidate alone is NVFP4, the integer candidate alone is NVINT4 up to where the E4M3 rounding falls
    c, s, a, e_fp, e_int = oracle.quantize(1, xb, threads=4, debug=True)
    assert abs(e_fp.astype(np.float64).sum() / xb.size * 1e3 - float(g["NVFP4"][0])) < 0.1
    assert abs(e_int.astype(np.float64).sum() / xb.size * 1e3 - float(g["NVINT4"][0])) < 0.1
    assert abs(np.minimum(e_fp, e_int).astype(np.float64).sum() / xb.size * 1e3 - float(g["IF4"][0])) < 0.1


def test_format_facts(oracle):
    g = read_golden("format_facts.txt")
    paper_fp4 = [float(v) for v in g["fp4_magnitudes"]]
    for fmt in (0, 1):
        vals = [float(oracle.fp_value(fmt, c)) for c in range(16)]
        assert vals[:8] == paper_fp4 and vals[8:] == [-v for v in paper_fp4]
        assert np.signbit(np.float32(vals[8]))
    assert float(oracle.m_fp(1)) == float(g["m_fp4"][0]) and float(oracle.m_int(1)) == float(g["int4_max"][0])
    assert float(oracle.e4m3_value(0x7E)) == float(g["m_fp8"][0])
    assert float(oracle.e4m3_value(0x7E)) * 6 == float(g["max_before_alpha"][0])
    assert float(oracle.e4m3_value(0x01)) * 0.5 == 2.0 ** float(g["min_before_alpha_log2"][0])
    for key, fmt in (("if4", 1), ("if3", 2), ("if6_e2m3", 3), ("if6_e3m2", 4)):
        num, den = (float(v) for v in g["post_factor_" + key])
        assert oracle.c_post(fmt) == np.float32(num) / np.float32(den)
        assert oracle.c_pre(fmt) == np.float32(den) / np.float32(num)
        assert float(oracle.m_fp(fmt)) == num and float(oracle.m_int(fmt)) == den
    for key, fmt in (("if3", 2), ("if4", 1), ("nvfp4", 0), ("if6", 3), ("if6", 4)):
        bpp = (oracle.codes_bytes(fmt, 1, 16) + oracle.scales_bytes(1, 16)) * 8 / 16
        assert bpp == float(g["bits_per_param_" + key][0])


def test_philox_known_answers(oracle):
    with open(os.path.join(GOLD, "philox4x32_10_kat.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(v, 16) for v in r]
        assert oracle.philox4x32_10(w[0:4], w[4:6]) == w[6:10]


# --------------------------------------------------------------------------- grids and conversions

@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_fp_grid_matches_definition(oracle, fmt):
    g = fp_grid(fmt)
    b = oracle.fmt_bits(fmt)
    assert len(g) == 1 << (b - 1) and g[-1] == float(oracle.m_fp(fmt))
    for c, v in enumerate(g):
        assert float(oracle.fp_value(fmt, c)) == v
        assert float(oracle.fp_value(fmt, c | (1 << (b - 1)))) == -v
        assert oracle.fp_encode(fmt, v) == c                      # representable values round-trip
        assert oracle.fp_encode(fmt, -float(v)) == (c | (1 << (b - 1)))  # sign kept, also for -0


@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_fp_encode_nearest_ties_even_saturating(oracle, fmt):
    g = np.array(fp_grid(fmt))
    rng = np.random.default_rng(7)
    ys = list(rng.uniform(-1.2 * g[-1], 1.2 * g[-1], 3000).astype(np.float32))
    mids = (g[:-1] + g[1:]) / 2
    for m in mids:  # exact midpoints and their float32 neighbours
        m32 = np.float32(m)
        assert float(m32) == m
        ys += [m32, np.nextafter(m32, np.float32(np.inf)), np.nextafter(m32, np.float32(-np.inf))]
    ys += [np.float32(g[-1] * 1.0001), np.float32(1e30), np.float32(-1e30), np.float32(1e-30)]
    for y in ys:
        code = oracle.fp_encode(fmt, y)
        mag = code & (len(g) - 1)
        a = min(abs(float(y)), g[-1])
        dist = np.abs(g - a)
        best = dist.min()
        assert dist[mag] == best
        ties = np.flatnonzero(dist == best)
        if len(ties) == 2:
            assert mag % 2 == 0
        assert (code >> (oracle.fmt_bits(fmt) - 1)) == int(np.signbit(y))


@pytest.mark.parametrize("fmt", IF_FMTS)
def test_int_candidate_rounds_the_exact_product_once(oracle, fmt):
    """Step 7: k = nearest integer (ties to even) of the real product y * fp32(M_INT/M_FP), clamped.
    Checked in exact rational arithmetic on every bf16 y in range, on random float32 y, and on values
    built to sit next to a half-integer product."""
    from fractions import Fraction
    c = Fraction(float(oracle.c_pre(fmt)))
    top = int(oracle.m_int(fmt))
    mfp = float(oracle.m_fp(fmt))

    def exact(y):
        p = Fraction(float(y)) * c
        k = int(p.numerator // p.denominator)          # floor
        frac = p - k
        if frac > Fraction(1, 2) or (frac == Fraction(1, 2) and k % 2 == 1):
            k += 1
        return max(-top, min(top, k))

    ys = [v for v in I.bf16_bits_to_f32(np.arange(0x3C00, 0x4100, dtype=np.uint16)) if abs(v) <= 1.3 * mfp]
    rng = np.random.default_rng(77)
    ys += list(rng.uniform(-1.3 * mfp, 1.3 * mfp, 3000).astype(np.float32))
    for k in range(-top - 2, top + 2):                   # neighbours of every half-integer product
        y0 = np.float32((k + 0.5) / float(c))
        for _ in range(4):
            ys += [y0, -y0]
            y0 = np.nextafter(y0, np.float32(np.inf))
        y0 = np.float32((k + 0.5) / float(c))
        for _ in range(4):
            y0 = np.nextafter(y0, np.float32(-np.inf))
            ys.append(y0)
    for y in ys:
        assert oracle.int_encode(fmt, y) == exact(y), (fmt, float(y))


def test_e4m3_matches_torch_cast(oracle):
    """In range, the scale rounding is torch's float8_e4m3fn cast (nearest, ties to even)."""
    torch = pytest.importorskip("torch")
    g = np.array(e4m3_grid())
    assert len(g) == 127 and g[-1] == 448.0
    for c, v in enumerate(g):
        assert float(oracle.e4m3_value(c)) == v and oracle.e4m3_encode(v) == c
    rng = np.random.default_rng(11)
    ts = list(np.exp(rng.uniform(np.log(2.0 ** -12), np.log(448.0), 4000)).astype(np.float32))
    for m in (g[:-1] + g[1:]) / 2:
        m32 = np.float32(m)
        ts += [m32, np.nextafter(m32, np.float32(np.inf)), np.nextafter(m32, np.float32(0))]
    ts = np.array(ts, dtype=np.float32)
    want = torch.from_numpy(ts).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([oracle.e4m3_encode(t) for t in ts], dtype=np.uint8)
    assert np.array_equal(got, want)
    # saturation above 448 (torch's cast does not saturate, so this part is by definition)
    for t in (448.0, 449.0, 464.0, 480.0, 1e9, np.inf):
        assert oracle.e4m3_encode(np.float32(t)) == 0x7E
    assert oracle.e4m3_encode(np.float32(2.0 ** -10)) == 0       # tie between 0 and 2^-9 -> even code 0
    assert oracle.e4m3_encode(np.nextafter(np.float32(2.0 ** -10), np.float32(1))) == 1
    assert np.isnan(oracle.e4m3_value(0x7F))


def test_bf16_rounding_matches_torch(oracle):
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(5)
    v = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    u = v.view(np.uint32).copy()
    u[:5000] = (u[:5000] & 0xFFFF0000) | 0x8000           # exact ties
    v = u.view(np.float32)
    want = torch.from_numpy(v.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.f32_to_bf16(x) for x in v], dtype=np.uint16)
    assert np.array_equal(got, want)
    assert np.array_equal(I.f32_to_bf16_bits(v), want)


def test_pack_is_little_endian_bitstream(oracle):
    """Each element placed alone: its code must appear at bits [b*j, b*j+b)."""
    for fmt in ALL_FMTS:
        b = oracle.fmt_bits(fmt)
        top = float(oracle.m_fp(fmt))
        for j in range(16):
            x = np.zeros((1, 16), np.float32)
            x[0, j] = -top
            c, s, a = oracle.quantize(fmt, I.f32_to_bf16_bits(x), flags=oracle.F_ALPHA_GIVEN, alpha=2.0 ** -8)
            codes = unpack_bitstream(c[0], b)
            assert np.count_nonzero(codes) == 1 and codes[j] != 0
            val = oracle.dequantize(fmt, c, s, 2.0 ** -8, 1, 16, out_fp32=True)
            assert val[0, j] == -top and np.count_nonzero(val) == 1


# --------------------------------------------------------------------------- invariants on random tensors

def _cases():
    cases = {
        "cfg1": I.generate("cfg1", 64, 256),
        "cfg2": I.generate("cfg2", 48, 1024),
        "cfg3": I.generate("cfg3a", 32, 512),
        "cfg4": I.generate("cfg4", 64, 256),
        "cfg5": I.generate("cfg5", 64, 512),
    }
    cases.update(I.edge_tensors())
    return cases


CASES = _cases()


@pytest.mark.parametrize("fmt", IF_FMTS)
@pytest.mark.parametrize("case", sorted(CASES))
def test_selection_invariants(oracle, fmt, case):
    xb = CASES[case]
    rows, cols = xb.shape
    c, s, a, efp, eint = oracle.quantize(fmt, xb, debug=True)
    flag = (s >> 7).astype(bool)
    # chosen error <= other error; integer only if strictly smaller (step 10)
    assert np.all(eint[flag] < efp[flag])
    assert np.all(~(eint[~flag] < efp[~flag]))
    # the byte 0x80 ("minus zero scale") never appears; zero scale means all-zero codes
    assert not np.any(s == 0x80)
    b = oracle.fmt_bits(fmt)
    cg = c.reshape(rows, cols // 16, 2 * b)
    assert not np.any(cg[s == 0])
    # the most negative integer pattern is never produced
    for r in range(rows):
        codes = unpack_bitstream(c[r], b).reshape(-1, 16)
        assert not np.any(codes[flag[r]] == (1 << (b - 1)))


@pytest.mark.parametrize("case", sorted(CASES))
def test_fp_groups_are_nvfp4_groups(oracle, case):
    """Sign-bit semantics (Sec. 3): a group with flag 0 is byte for byte the NVFP4 group."""
    xb = CASES[case]
    rows, cols = xb.shape
    c4, s4, a4 = oracle.quantize(1, xb)
    cn, sn, an = oracle.quantize(0, xb)
    assert a4 == an
    assert np.array_equal(s4 & 0x7F, sn) and not np.any(sn & 0x80)
    keep = (s4 >> 7) == 0
    g4 = c4.reshape(rows, cols // 16, 8)
    gn = cn.reshape(rows, cols // 16, 8)
    assert np.array_equal(g4[keep], gn[keep])


@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_bruteforce_elements_and_flag(oracle, fmt):
    """For the scale the oracle chose, every stored code is (up to float32 near-ties) the
    closest grid point to the input, and the flag is the arg-min of the two squared errors,
    all checked in float64 over every code of the grid."""
    rng = np.random.default_rng(100 + fmt)
    b = oracle.fmt_bits(fmt)
    g = np.array(fp_grid(fmt))
    fpvals = np.concatenate([g, -g])
    mint = int(oracle.m_int(fmt))
    ivals = np.arange(-mint, mint + 1, dtype=np.float64) if fmt else None
    for trial, case in enumerate(("cfg1", "cfg2", "cfg5", "wide_dynamic_range")):
        xb = CASES[case][:8, :128]
        rows, cols = xb.shape
        xf = I.bf16_bits_to_f32(xb).astype(np.float64)
        c, s, a = oracle.quantize(fmt, xb)
        for r in range(rows):
            codes = unpack_bitstream(c[r], b).reshape(-1, 16)
            for gi in range(cols // 16):
                sb = int(s[r, gi])
                x = xf[r, gi * 16:(gi + 1) * 16]
                if sb == 0:
                    assert not codes[gi].any()
                    continue
                d = float(np.float32(oracle.e4m3_value(sb)) * np.float32(a))
                best_fp = np.abs(fpvals[None, :] * d - x[:, None]).min(axis=1)
                slack = 1e-6 * np.abs(x) + 1e-30
                if sb >> 7:
                    d_i = float(np.float32(d) * oracle.c_post(fmt))
                    k = codes[gi].astype(np.int64)
                    k = np.where(k >= (1 << (b - 1)), k - (1 << b), k)
                    err = np.abs(k * d_i - x)
                    best_i = np.abs(ivals[None, :] * d_i - x[:, None]).min(axis=1)
                    assert np.all(err <= best_i + slack)
                    assert (err ** 2).sum() <= (best_fp ** 2).sum() * (1 + 1e-5) + 1e-60
                else:
                    v = fpvals[(codes[gi] & (len(g) - 1)) + len(g) * (codes[gi] >> (b - 1))]
                    err = np.abs(v * d - x)
                    assert np.all(err <= best_fp + slack)
                    if fmt:
                        d_i = float(np.float32(d) * oracle.c_post(fmt))
                        best_i = np.abs(ivals[None, :] * d_i - x[:, None]).min(axis=1)
                        assert (err ** 2).sum() <= (best_i ** 2).sum() * (1 + 1e-5) + 1e-60


def test_tie_goes_to_fp(oracle):
    """One outlier, everything else rounding to zero in both encodings: equal errors -> FP."""
    x = np.zeros((1, 16), np.float32)
    x[0, 3] = 6.0
    x[0, 7] = 0.0625     # rounds to 0 in both candidates; same error either way
    c, s, a, efp, eint = oracle.quantize(1, I.f32_to_bf16_bits(x), flags=oracle.F_ALPHA_GIVEN, alpha=2.0 ** -8,
                                         debug=True)
    assert efp[0, 0] == eint[0, 0] and s[0, 0] >> 7 == 0


def test_fp4_midpoints_round_to_even(oracle):
    xb = I.edge_tensors()["fp4_midpoints"]
    c, s, a = oracle.quantize(0, xb, flags=oracle.F_ALPHA_GIVEN, alpha=2.0 ** -8)   # Delta = 256 * 2^-8... d = 1
    assert np.all(s == oracle.e4m3_encode(np.float32(256.0)))
    codes = unpack_bitstream(c[0], 4)[:16]
    want_mag = [0, 1, 1, 2, 2, 4, 4, 6]          # values after nearest-even on the paper's grid
    vals = [fp_grid(0)[k & 7] * (-1 if k >> 3 else 1) for k in codes]
    assert vals == want_mag + [-v for v in want_mag]
    assert all(k >> 3 == 1 for k in codes[8:])   # sign kept, "-0.25 -> -0" included


# --------------------------------------------------------------------------- round trips and scaling

@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_fp_round_trip_of_representable_tensor(oracle, fmt):
    """Tensors built from (alpha = 2^k, scale bytes, FP codes) whose groups contain +-M_FP and
    whose largest scale is 448 quantize back to the same bytes and dequantize exactly."""
    rng = np.random.default_rng(40 + fmt)
    b = oracle.fmt_bits(fmt)
    g = np.array(fp_grid(fmt))
    rows, gpr = 6, 5
    alpha = np.float32(2.0 ** -3)
    sb = rng.integers(0x20, 0x7E, size=(rows, gpr))    # normal-range scales, at least 2 binades below the top
    sb[2, 1] = 0x7E
    mag = rng.integers(0, len(g), size=(rows, gpr, 16))
    sign = rng.integers(0, 2, size=(rows, gpr, 16))
    mag[:, :, 0] = len(g) - 1                          # every group holds +-M_FP -> gmax fixes the scale
    delta = np.array([[float(oracle.e4m3_value(int(v))) for v in row] for row in sb])
    x = (np.where(sign == 1, -1.0, 1.0) * g[mag]) * delta[:, :, None] * float(alpha)
    xb = I.f32_to_bf16_bits(x.reshape(rows, gpr * 16).astype(np.float32))
    if fmt in (0, 1, 2):   # <= 2+4 significant bits: exactly representable in bf16
        assert np.array_equal(I.bf16_bits_to_f32(xb).astype(np.float64), x.reshape(rows, -1))
    fmt_fp_only = 0 if fmt in (0, 1) else fmt
    c, s, a = oracle.quantize(fmt_fp_only, xb)
    assert a == alpha
    if fmt in (0, 1, 2):
        assert np.array_equal(s & 0x7F, sb.astype(np.uint8))
    out = oracle.dequantize(fmt_fp_only, c, s, a, rows, gpr * 16)
    if fmt in (0, 1, 2):
        flagged = (s >> 7).astype(bool)
        back = I.bf16_bits_to_f32(out).reshape(rows, gpr, 16)
        assert np.array_equal(back[~flagged], I.bf16_bits_to_f32(xb).reshape(rows, gpr, 16)[~flagged])
        if fmt == 0:
            for r in range(rows):
                codes = unpack_bitstream(c[r], b).reshape(gpr, 16)
                nz = mag[r] != 0   # the sign of a zero is kept too, so compare all
                assert np.array_equal(codes, mag[r] | (sign[r] << (b - 1)))


def test_int_round_trip(oracle):
    """Groups k * 6 * 2^j with k in -7..7 and a 7 present: Delta = 7 * 2^j', d * 6/7 exact."""
    rng = np.random.default_rng(9)
    rows, gpr = 4, 6
    k = rng.integers(-7, 8, size=(rows, gpr, 16))
    k[:, :, 5] = 7
    k[:, :, 6] = -6          # makes FP4 strictly worse: 36 -> 5.14 not on the FP grid
    x = (k * 6.0).astype(np.float32).reshape(rows, gpr * 16)
    xb = I.f32_to_bf16_bits(x)
    assert np.array_equal(I.bf16_bits_to_f32(xb), x)
    c, s, a, efp, eint = oracle.quantize(1, xb, debug=True)
    assert a == np.float32(42.0 / 2688.0)
    assert np.all(s >> 7 == 1) and np.all(eint == 0)
    back = I.bf16_bits_to_f32(oracle.dequantize(1, c, s, a, rows, gpr * 16))
    assert np.array_equal(back, x)
    for r in range(rows):
        codes = unpack_bitstream(c[r], 4).reshape(gpr, 16)
        assert np.array_equal(codes, k[r] & 0xF)


@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_power_of_two_rescaling(oracle, fmt):
    """Multiplying the tensor by 2^k leaves codes and scale bytes unchanged and scales alpha."""
    xb = CASES["cfg5"][:16, :256]
    x = I.bf16_bits_to_f32(xb)
    c0, s0, a0 = oracle.quantize(fmt, xb)
    for k in (-20, 7, 30):
        xk = I.f32_to_bf16_bits(x * np.float32(2.0 ** k))
        c, s, a = oracle.quantize(fmt, xk)
        assert a == a0 * np.float32(2.0 ** k)
        assert np.array_equal(c, c0) and np.array_equal(s, s0)


@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_dequantize_error_bound(oracle, fmt):
    """|dequant - x| never exceeds half the coarsest step of the chosen grid (plus bf16 rounding)."""
    xb = CASES["cfg2"]
    rows, cols = xb.shape
    xf = I.bf16_bits_to_f32(xb).astype(np.float64)
    c, s, a = oracle.quantize(fmt, xb)
    d = oracle.dequantize(fmt, c, s, a, rows, cols, out_fp32=True).astype(np.float64)
    delta = np.array([[float(oracle.e4m3_value(int(v))) for v in row] for row in s]) * float(a)
    g = np.array(fp_grid(fmt))
    fp_half_step = np.diff(g).max() / 2
    # scale rounding may shrink the range by 17/16, so the top value can clip by M_FP/16
    bound_fp = np.maximum(fp_half_step, g[-1] / 16) * delta
    bound_int = (0.5 * float(oracle.c_post(fmt)) + g[-1] / 16) * delta if fmt else bound_fp
    bound = np.where(s >> 7 == 1, bound_int, bound_fp)
    err = np.abs(d - xf).reshape(rows, cols // 16, 16).max(axis=2)
    ok = s & 0x7F >= 8                   # normal-range scales only; subnormal scales round coarsely
    assert np.all(err[ok] <= bound[ok] * (1 + 1e-6))


def test_all_zero_and_empty(oracle):
    z = np.zeros((3, 48), np.uint16)
    for fmt in ALL_FMTS:
        c, s, a = oracle.quantize(fmt, z)
        assert a == np.float32(1.0) and not c.any() and not s.any()
        assert not oracle.dequantize(fmt, c, s, a, 3, 48).any()
        c, s, a = oracle.quantize(fmt, np.zeros((0, 64), np.uint16))
        assert c.size == 0 and s.size == 0


def test_threads_do_not_change_result(oracle):
    xb = CASES["cfg5"]
    a1 = oracle.quantize(1, xb, threads=1)
    a4 = oracle.quantize(1, xb, threads=4)
    assert all(np.array_equal(p, q) for p, q in zip(a1, a4))
    d1 = oracle.dequantize(1, *a1, *xb.shape, threads=1)
    d4 = oracle.dequantize(1, *a1, *xb.shape, threads=3)
    assert np.array_equal(d1, d4)


# --------------------------------------------------------------------------- Hadamard option

def test_hadamard_matches_dense_matrix(oracle):
    scipy_linalg = pytest.importorskip("scipy.linalg")
    H = scipy_linalg.hadamard(16).astype(np.float64)    # natural-order Sylvester matrix
    rng = np.random.default_rng(3)
    for mask in (0x0000, 0xFFFF, 0x1234, oracle.hadamard_sign_mask(5)):
        sgn = np.array([-1.0 if (mask >> i) & 1 else 1.0 for i in range(16)])
        x = rng.integers(-64, 65, 16).astype(np.float32)   # small integers: every partial sum is exact
        want = 0.25 * (H @ (sgn * x))
        assert np.array_equal(oracle.hadamard16(x, mask).astype(np.float64), want)
        # H (H x) / 16 = x : applying it twice with s = +1 is the identity on exact data
        once = oracle.hadamard16(x, 0)
        assert np.array_equal(oracle.hadamard16(once, 0), x)
        # Parseval: the transform keeps the sum of squares
        y = oracle.hadamard16(x, mask).astype(np.float64)
        assert np.isclose((y ** 2).sum(), (x.astype(np.float64) ** 2).sum())


def test_hadamard_quantize_equals_quantize_of_transformed(oracle):
    """With data on which the transform is exact in bf16, the fused option equals transforming first."""
    rng = np.random.default_rng(12)
    mask = 0xA5C3
    x = rng.integers(-8, 9, (8, 64)).astype(np.float32)
    xt = np.concatenate([oracle.hadamard16(x[r, c:c + 16], mask) for r in range(8) for c in range(0, 64, 16)])
    xt = xt.reshape(8, 64)
    xtb = I.f32_to_bf16_bits(xt)
    assert np.array_equal(I.bf16_bits_to_f32(xtb), xt)           # |values| <= 32 in steps of 1/4: exact in bf16?
    got = oracle.quantize(1, I.f32_to_bf16_bits(x), flags=oracle.F_HADAMARD16, sign_mask=mask)
    want = oracle.quantize(1, xtb)
    assert all(np.array_equal(p, q) for p, q in zip(got, want))


# --------------------------------------------------------------------------- stochastic rounding

def test_sr_uniform_fields(oracle):
    seed = 0x0123456789ABCDEF
    for base in (0, 8, 1 << 35):
        w = oracle.philox4x32_10([(base >> 3) & 0xFFFFFFFF, (base >> 3) >> 32, 0, 0],
                                 [seed & 0xFFFFFFFF, seed >> 32])
        for j in range(8):
            h = (w[j >> 1] >> (16 * (j & 1))) & 0xFFFF
            assert oracle.sr_uniform(seed, base + j) == np.float32((h + 0.5) / 65536.0)


def test_sr_keeps_representable_and_brackets(oracle):
    """SR leaves representable values alone and otherwise returns one of the two neighbours."""
    rng = np.random.default_rng(21)
    x = rng.uniform(-6, 6, (8, 64)).astype(np.float32)
    x[:, 0::16] = 6.0                      # every group holds the maximum, so d = 1 everywhere
    x[:, 1:9] = [0, 0.5, 1, 1.5, 2, 3, 4, -6]
    xb = I.f32_to_bf16_bits(x)
    xf = I.bf16_bits_to_f32(xb).astype(np.float64)
    g = np.array(fp_grid(0))
    allv = np.sort(np.concatenate([-g[1:], g]))
    for seed in range(5):
        c, s, a = oracle.quantize(0, xb, flags=oracle.F_STOCHASTIC | oracle.F_ALPHA_GIVEN, alpha=2.0 ** -8,
                                  sr_seed=seed)
        d = oracle.dequantize(0, c, s, 2.0 ** -8, 8, 64, out_fp32=True).astype(np.float64)
        assert np.array_equal(d[:, 0:9], xf[:, 0:9])
        lo = allv[np.searchsorted(allv, xf, side="right") - 1]
        hi = allv[np.minimum(np.searchsorted(allv, xf, side="left"), len(allv) - 1)]
        assert np.all((d == lo) | (d == hi))


@pytest.mark.parametrize("fmt", [0, 2, 3, 4])
def test_sr_index_probability_is_the_fractional_position(oracle, fmt):
    """App. B: a value between grid points lo < a < hi rounds up with probability (a-lo)/(hi-lo), and a
    grid point stays put.  Counted over evenly spaced values of the 16-bit uniform; built from the grid
    alone (searchsorted), not from the oracle's own bracket search."""
    g = np.array(fp_grid(fmt), dtype=np.float64)
    us = ((np.arange(65536) + 0.5) / 65536.0).astype(np.float32)[::16]      # 4096 evenly spaced draws
    rng = np.random.default_rng(100 + fmt)
    samples = list(g) + [float(np.float32(v)) for v in rng.uniform(0, g[-1], 40)]
    samples += [float(g[-1]) * 1.5, float(g[1]) * 0.25, float(g[-2] + g[-1]) / 2]
    for a in samples:
        idx = np.array([oracle.fp_sr(fmt, a, float(u)) for u in us])
        ac = min(a, g[-1])
        lo = int(np.searchsorted(g, ac, side="right") - 1)
        if g[lo] == ac:
            assert np.all(idx == lo), (fmt, a)
            continue
        assert set(np.unique(idx)) <= {lo, lo + 1}
        p = (ac - g[lo]) / (g[lo + 1] - g[lo])
        assert abs((idx == lo + 1).mean() - p) <= 1.0 / 4096 + 1e-9, (fmt, a, p)
        assert np.array_equal(idx == lo + 1, us.astype(np.float64) < p)     # "u < p" itself


def test_sr_int_candidate_probability(oracle):
    """The integer candidate under SR: floor or ceil of y*7/6, up with probability frac, clamped to +-7.
    Read back from the codes of groups the selection gives to the integer grid."""
    rows, cols = 1, 16
    for y_target in (0.3, 2.25, -4.6, 5.9, -6.0):
        z = y_target * 7.0 / 6.0
        ups = 0
        n = 0
        for seed in range(400):
            x = np.zeros((rows, cols), np.float32)
            x[0, :] = [6, 6 * 5 / 7, 6 * 3 / 7, 6 * 1 / 7, -6 * 5 / 7, -6 * 3 / 7, 0, 0, 0, 0, 0, 0, 0, 0, 0, y_target]
            xb = I.f32_to_bf16_bits(x)
            yb = float(I.bf16_bits_to_f32(xb)[0, 15])
            zb = yb * 7.0 / 6.0
            c, s, a = oracle.quantize(1, xb, flags=oracle.F_STOCHASTIC | oracle.F_ALPHA_GIVEN, alpha=1.0 / 64,
                                      sr_seed=seed)
            if not (s[0, 0] & 0x80):
                continue
            code = (int(c[0, 7]) >> 4) & 0xF
            k = code - 16 if code >= 8 else code
            assert k in (int(np.floor(zb)), int(np.ceil(zb))), (y_target, k)
            ups += k == int(np.ceil(zb))
            n += 1
        assert n > 100
        frac = zb - np.floor(zb)
        if frac > 0:
            assert abs(ups / n - frac) < 4.5 * np.sqrt(frac * (1 - frac) / n) + 1e-3, (y_target, ups / n, frac)


def test_sr_bias_signature(oracle):
    """App. B: NVFP4 with stochastic rounding is unbiased; IF4's selection on the stochastic
    candidates pushes near-maximal values slightly up.  Checked with the 17/16 scale option on
    (nothing clips) as an average over seeds."""
    xb = I.generate("cfg4", 32, 256)
    flags = oracle.F_HADAMARD16 | oracle.F_STOCHASTIC | oracle.F_SR_SCALE_17_16
    mask = oracle.hadamard_sign_mask(77)
    rows, cols = xb.shape
    xt = np.stack([oracle.hadamard16(I.bf16_bits_to_f32(xb)[r, c:c + 16], mask)
                   for r in range(rows) for c in range(0, cols, 16)]).reshape(rows, cols).astype(np.float64)
    n = 200
    mean = {0: np.zeros_like(xt), 1: np.zeros_like(xt)}
    for seed in range(n):
        for fmt in (0, 1):
            c, s, a = oracle.quantize(fmt, xb, flags=flags, sign_mask=mask, sr_seed=seed)
            mean[fmt] += oracle.dequantize(fmt, c, s, a, rows, cols, out_fp32=True)
    gmax = np.abs(xt).reshape(rows, cols // 16, 16).max(axis=2, keepdims=True)
    rel = (np.abs(xt).reshape(rows, cols // 16, 16) / gmax)
    sgn = np.sign(xt).reshape(rows, cols // 16, 16)
    for fmt in (0, 1):
        bias = ((mean[fmt] / n - xt).reshape(rows, cols // 16, 16) * sgn) / gmax   # outward bias, in units of gmax
        top = bias[rel > 0.9].mean()
        mid = bias[(rel > 0.2) & (rel < 0.6)].mean()
        if fmt == 0:
            assert abs(top) < 4e-3 and abs(mid) < 2e-3, (top, mid)
        else:
            assert top > 4e-3, top          # near-maximal values grow
            assert abs(mid) < 4e-3, mid


def test_sr_scale_option_prevents_clipping(oracle):
    """Without the 17/16 option an E4M3 scale rounded down lets |y| exceed M_FP, and the group
    maximum is clipped (negative bias); with it every |y| <= M_FP for normal-range scales."""
    xb = I.generate("cfg1", 64, 256)
    xf = I.bf16_bits_to_f32(xb).astype(np.float64)
    for opt, expect_clip in ((0, True), (oracle.F_SR_SCALE_17_16, False)):
        c, s, a = oracle.quantize(0, xb, flags=oracle.F_STOCHASTIC | opt, sr_seed=3)
        d = np.array([[float(oracle.e4m3_value(int(v))) for v in row] for row in s]) * float(a)
        ymax = (np.abs(xf).reshape(64, 16, 16).max(axis=2) / d)
        assert (ymax.max() > 6.0 * (1 + 1e-6)) == expect_clip
        if not expect_clip:
            assert ymax[s >= 8].max() <= 6.0 * (1 + 1e-6)


# --------------------------------------------------------------------------- block size 8 (Sec. 5.1, Table 5)

BS8 = {5: 0, 6: 1, 7: 2}          # block-size-8 format -> its 16-value sibling


def test_bs8_bits_per_parameter(oracle):
    g = read_golden("format_facts.txt")
    for key, fmt in (("if3_bs8", 7), ("if4_bs8", 6), ("nvfp4_bs8", 5)):
        bpp = (oracle.codes_bytes(fmt, 1, 16) + oracle.scales_bytes(1, 16, fmt)) * 8 / 16
        assert bpp == float(g["bits_per_param_" + key][0])
        assert oracle.fmt_group(fmt) == 8 and oracle.fmt_bits(fmt) == oracle.fmt_bits(BS8[fmt])


@pytest.mark.parametrize("fmt", sorted(BS8))
def test_bs8_equals_16_on_duplicated_halves(oracle, fmt):
    """A block whose two halves are identical: the 16-value format's single scale, flag and codes must
    equal the two (identical) groups of the block-size-8 format -- the sum of 16 squared errors is then
    exactly twice the sum of 8, so even the selection agrees.  Links BS8 to the pinned 16-value path."""
    half = CASES["cfg5"][:24, :256].reshape(24, 32, 8)
    xb = np.concatenate([half, half], axis=2).reshape(24, 512)
    c8, s8, a8 = oracle.quantize(fmt, xb)
    c16, s16, a16 = oracle.quantize(BS8[fmt], xb)
    assert a8 == a16
    assert np.array_equal(c8, c16)
    assert np.array_equal(s8[:, 0::2], s16) and np.array_equal(s8[:, 1::2], s16)
    d8 = oracle.dequantize(fmt, c8, s8, a8, 24, 512)
    assert np.array_equal(d8, oracle.dequantize(BS8[fmt], c16, s16, a16, 24, 512))


@pytest.mark.parametrize("fmt", [6, 7])
@pytest.mark.parametrize("case", ["cfg1", "cfg2", "cfg4", "wide_dynamic_range", "tiny_row", "zeros_3x48"])
def test_bs8_selection_invariants(oracle, fmt, case):
    xb = CASES[case]
    rows, cols = xb.shape
    c, s, a, efp, eint = oracle.quantize(fmt, xb, debug=True)
    assert s.shape == (rows, cols // 8)
    flag = (s >> 7).astype(bool)
    assert np.all(eint[flag] < efp[flag]) and np.all(~(eint[~flag] < efp[~flag]))
    assert not np.any(s == 0x80)
    # FP groups are the FP-only format's groups, byte for byte
    cn, sn, an = oracle.quantize(5 if fmt == 6 else fmt, xb)
    if fmt == 6:
        assert an == a and np.array_equal(s & 0x7F, sn)
        b = 4
        g4 = c.reshape(rows, cols // 8, b)
        gn = cn.reshape(rows, cols // 8, b)
        assert np.array_equal(g4[~flag], gn[~flag])


@pytest.mark.parametrize("fmt", sorted(BS8))
def test_bs8_bruteforce_elements(oracle, fmt):
    """Every stored code is (up to float32 near-ties) the closest grid point for the group's scale."""
    xb = CASES["cfg5"][:8, :128]
    rows, cols = xb.shape
    b = oracle.fmt_bits(fmt)
    g = np.array(fp_grid(BS8[fmt]))
    fpvals = np.concatenate([g, -g])
    mint = int(oracle.m_int(fmt))
    xf = I.bf16_bits_to_f32(xb).astype(np.float64)
    c, s, a = oracle.quantize(fmt, xb)
    for r in range(rows):
        codes = unpack_bitstream(c[r], b).reshape(-1, 8)
        for gi in range(cols // 8):
            sb = int(s[r, gi])
            x = xf[r, gi * 8:(gi + 1) * 8]
            if sb == 0:
                assert not codes[gi].any()
                continue
            d = float(np.float32(oracle.e4m3_value(sb)) * np.float32(a))
            slack = 1e-6 * np.abs(x) + 1e-30
            if sb >> 7:
                d_i = float(np.float32(d) * oracle.c_post(fmt))
                k = codes[gi].astype(np.int64)
                k = np.where(k >= (1 << (b - 1)), k - (1 << b), k)
                best = np.abs(np.arange(-mint, mint + 1)[None, :] * d_i - x[:, None]).min(axis=1)
                assert np.all(np.abs(k * d_i - x) <= best + slack)
            else:
                v = fpvals[(codes[gi] & (len(g) - 1)) + len(g) * (codes[gi] >> (b - 1))]
                best = np.abs(fpvals[None, :] * d - x[:, None]).min(axis=1)
                assert np.all(np.abs(v * d - x) <= best + slack)


def test_bs8_has_lower_error_than_16(oracle):
    """Finer scales cannot be worse on N(0,1): the ordering behind Table 5's BS8 rows."""
    xb = I.generate("cfg1", 256, 1024)
    xf = I.bf16_bits_to_f32(xb).astype(np.float64)
    for f8, f16 in BS8.items():
        mse = {}
        for f in (f8, f16):
            c, s, a = oracle.quantize(f, xb, threads=4)
            mse[f] = np.mean((oracle.dequantize(f, c, s, a, 256, 1024, out_fp32=True, threads=4) - xf) ** 2)
        assert mse[f8] < 0.85 * mse[f16], (f8, mse)


# --------------------------------------------------------------------------- tensor-core scale layout

def test_swizzled_scale_layout_definition(oracle):
    """The 128x4-tile layout against its closed-form byte offset, on shapes with ragged tiles."""
    for rows, k in ((128, 4), (300, 13), (1, 1), (257, 64)):
        s = (np.arange(rows * k, dtype=np.int64) * 7 % 251 + 1).astype(np.uint8).reshape(rows, k)
        out = oracle.swizzle_scales(s, fill=0)
        kt = -(-k // 4)
        assert out.size == -(-rows // 128) * kt * 512
        seen = np.zeros(out.size, bool)
        for r in range(rows):
            for c in range(k):
                off = ((r // 128) * kt + c // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + c % 4
                assert out[off] == s[r, c]
                seen[off] = True
        assert not out[~seen].any()                      # padding untouched
        # one 512-byte tile holds exactly rows 128t..128t+127 x scales 4u..4u+3
        tile0 = out[:512]
        want = set(s[:128, :4].reshape(-1).tolist()) | {0}
        assert set(tile0.tolist()) <= want


# --------------------------------------------------------------------------- MAC semantics (Sec. 5.2)

def test_split_dequantize_recombines(oracle):
    """FP-group part + (M_FP/M_INT) * raw integer-group part == the ordinary dequantization, and both
    parts are exactly representable in bf16 (a 4-bit code times a 4-bit-mantissa scale)."""
    xb = CASES["cfg5"]
    rows, cols = xb.shape
    c, s, a = oracle.quantize(1, xb)
    full = oracle.dequantize(1, c, s, 1.0, rows, cols, out_fp32=True).astype(np.float64)
    fp = oracle.dequantize(1, c, s, 1.0, rows, cols, out_fp32=True, select=oracle.F_FP_GROUPS_ONLY)
    it = oracle.dequantize(1, c, s, 1.0, rows, cols, out_fp32=True, select=oracle.F_INT_GROUPS_RAW)
    flag = np.repeat((s >> 7).astype(bool), 16, axis=1)
    assert not fp[flag].any() and not it[~flag].any()
    assert np.array_equal(fp[~flag].astype(np.float64), full[~flag])
    assert np.allclose(it[flag].astype(np.float64) * (6.0 / 7.0), full[flag], rtol=1e-6)
    for part in (fp, it):
        assert np.array_equal(I.bf16_bits_to_f32(I.f32_to_bf16_bits(part)), part)


def test_mac_constants_and_reference(oracle):
    """Sec. 5.2: 6/7 for one integer operand, 36/49 for two.  On a tiny case the reference equals the
    dot product of the ordinary dequantized operands (same real number, different rounding)."""
    g = read_golden("format_facts.txt")
    one = float(g["mac_rescale_one_int"][0]) / float(g["mac_rescale_one_int"][1])
    two = float(g["mac_rescale_two_int"][0]) / float(g["mac_rescale_two_int"][1])
    assert abs(one * one - two) < 1e-15
    a = I.generate("cfg1", 32, 256)
    b = I.generate("cfg5", 48, 256)
    qa, qb = oracle.quantize(1, a), oracle.quantize(1, b)
    ref = oracle.mac_matmul_reference(1, qa, qb, 32, 48, 256)
    da = oracle.dequantize(1, *qa, 32, 256, out_fp32=True).astype(np.float64)
    db = oracle.dequantize(1, *qb, 48, 256, out_fp32=True).astype(np.float64)
    assert np.abs(ref - da @ db.T).max() <= 1e-5 * np.abs(ref).max()    # cancellation: compare on the result's scale


# --------------------------------------------------------------------------- dequantize on arbitrary bytes

BASE_FMT = {0: 0, 1: 1, 2: 2, 3: 3, 4: 4, 5: 0, 6: 1, 7: 2}       # block-size-8 variants share their sibling's element format


def dequantize_by_definition(oracle, fmt, codes, scales, alpha, rows, cols):
    """Sec. 3 and Sec. 4.1 written out with numpy and library casts, for ANY byte values:
    element = value(code) * Delta * alpha, times M_FP / M_INT for an integer group, product in FP32, then BF16.
      - Delta: torch's float8_e4m3fn decode of the scale byte's low seven bits (0x7F is NaN by that format);
      - the group is an integer group iff the format has an integer alternative and bit 7 of the byte is set
        (Sec. 3: the flag sits in the sign bit an NVFP4 scale leaves unused, so plain NVFP4 ignores it);
      - FP codes: sign | index into the format's magnitude grid; integer codes: two's complement in b bits
        (Sec. 3 footnote: the most negative pattern is given up by the encoder, the decoder still reads it);
      - BF16 rounding: torch's cast."""
    torch = pytest.importorskip("torch")
    base = BASE_FMT[fmt]
    b, G = oracle.fmt_bits(fmt), oracle.fmt_group(fmt)
    has_int = base != 0
    e4 = torch.arange(128, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy()
    grid = np.array(fp_grid(base), dtype=np.float32)
    code = np.stack([unpack_bitstream(row, b) for row in np.asarray(codes).reshape(rows * cols // 16, 2 * b)])
    code = code.reshape(rows, cols).astype(np.int64)
    sb = np.repeat(np.asarray(scales, dtype=np.uint8).reshape(rows, cols // G), G, axis=1).astype(np.int64)
    flag = (sb >> 7).astype(bool) if has_int else np.zeros_like(sb, dtype=bool)
    with np.errstate(invalid="ignore"):
        d = e4[sb & 0x7F] * np.float32(alpha)
        if has_int:
            c_post = np.float32(oracle.m_fp(fmt)) / np.float32(oracle.m_int(fmt))
            d = np.where(flag, d * c_post, d).astype(np.float32)
        v_fp = grid[code & ((1 << (b - 1)) - 1)] * np.where(code >> (b - 1), np.float32(-1), np.float32(1))
        v_int = np.where(code >= (1 << (b - 1)), code - (1 << b), code).astype(np.float32)
        out32 = (np.where(flag, v_int, v_fp).astype(np.float32) * d).astype(np.float32)
    bf = torch.from_numpy(out32.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    return out32, bf


def same_bits_or_both_nan(got, want, as_float):
    g, w = np.asarray(got), np.asarray(want)
    gn, wn = np.isnan(as_float(g)), np.isnan(as_float(w))
    return np.array_equal(gn, wn) and np.array_equal(g[~gn], w[~wn])


@pytest.mark.parametrize("fmt", [0, 1, 2, 3, 4, 5, 6, 7])
def test_dequantize_arbitrary_bytes_against_definition(oracle, fmt):
    """Bytes the quantizer never produces decode as the formats define them: scale 0x7F / 0xFF is the E4M3 NaN
    and propagates, 0x80 is a zero scale with the flag set, the most negative integer code is plain two's
    complement, the FP code 'minus zero' gives -0, and plain NVFP4 ignores bit 7 of its scale bytes."""
    rows, cols, alpha = 16, 1024, np.float32(0.0173)
    codes, scales = I.arbitrary_quantized_bytes(oracle.fmt_bits(fmt), oracle.fmt_group(fmt), rows, cols)
    want32, want16 = dequantize_by_definition(oracle, fmt, codes, scales, alpha, rows, cols)
    got32 = oracle.dequantize(fmt, codes, scales, alpha, rows, cols, out_fp32=True)
    got16 = oracle.dequantize(fmt, codes, scales, alpha, rows, cols)
    assert np.isnan(want32).any() and (want32 == 0).any()
    assert same_bits_or_both_nan(got32.view(np.uint32), want32.view(np.uint32), lambda u: u.view(np.float32))
    assert same_bits_or_both_nan(got16, want16, I.bf16_bits_to_f32)
    # the named cases, one by one (IF4): most negative code under an integer flag, -0 under an FP flag
    if fmt == 1:
        c = np.zeros((1, 8), np.uint8)
        c[0, 0] = 0x88                                              # nibbles 8, 8
        out = oracle.dequantize(1, c, np.array([[0xC8]], np.uint8), 1.0, 1, 16, out_fp32=True)   # flag | E4M3(4.0)
        assert out[0, 0] == np.float32(-8) * (np.float32(4) * (np.float32(6) / np.float32(7)))
        out = oracle.dequantize(1, c, np.array([[0x48]], np.uint8), 1.0, 1, 16, out_fp32=True)   # same byte, FP group
        assert out[0, 0] == 0 and np.signbit(out[0, 0])
        assert np.isnan(oracle.dequantize(1, c, np.array([[0xFF]], np.uint8), 1.0, 1, 16, out_fp32=True)).all()


# --------------------------------------------------------------------------- order of the error sums

def _round_to_f32(q):
    """Exact rational -> nearest binary32 (ties to even, subnormals kept) by integer arithmetic."""
    from fractions import Fraction
    if q == 0:
        return Fraction(0)
    sign, a = (-1 if q < 0 else 1), abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()        # 2^(e-1) <= a < 2^(e+1)
    if Fraction(2) ** e > a:
        e -= 1                                                        # now 2^e <= a < 2^(e+1)
    ulp = Fraction(2) ** (max(e, -126) - 23)
    n, rem = divmod(a, ulp)
    if rem * 2 > ulp or (rem * 2 == ulp and n % 2 == 1):
        n += 1
    return sign * n * ulp


def test_error_sum_order_is_four_fused_chains(oracle):
    """The selection compares SUM16 of the squared errors.  Its order -- four fused multiply-add chains over the
    elements {0,2,4,6}, {1,3,5,7}, {8,..,14}, {9,..,15}, then (S0 + S1) + (S2 + S3) -- is recomputed here in exact
    rational arithmetic with one explicit rounding per operation, from the stored codes of each group, and must equal
    the error the oracle reports for the chosen candidate bit for bit.  A plain left-to-right sum differs on many of
    the same groups, so this test fails for a sequential implementation."""
    from fractions import Fraction as Fr
    xb = I.generate("cfg1", 8, 256)
    rows, cols = xb.shape
    c, s, a, efp, eint = oracle.quantize(1, xb, debug=True)
    x = I.bf16_bits_to_f32(xb)
    e4, grid = e4m3_grid(), fp_grid(1)
    c_post = np.float32(6) / np.float32(7)
    differs_from_sequential = 0
    for r in range(rows):
        for g in range(cols // 16):
            sb = int(s[r, g])
            if (sb & 0x7F) == 0:
                continue
            flag = sb >> 7
            d = np.float32(e4[sb & 0x7F]) * np.float32(a)
            if flag:
                d = np.float32(d * c_post)
            codes = unpack_bitstream(c[r, 8 * g: 8 * g + 8], 4)
            errs = []
            for j in range(16):
                k = int(codes[j])
                v = (k - 16 if k >= 8 else k) if flag else (-1 if k & 8 else 1) * grid[k & 7]
                errs.append(_round_to_f32(Fr(v) * Fr(float(d)) - Fr(float(x[r, 16 * g + j]))))     # one fused rounding
            chains = []
            for first in (0, 1, 8, 9):
                acc = Fr(0)
                for j in range(first, first + 8, 2):
                    acc = _round_to_f32(errs[j] * errs[j] + acc)
                chains.append(acc)
            total = _round_to_f32(_round_to_f32(chains[0] + chains[1]) + _round_to_f32(chains[2] + chains[3]))
            reported = (eint if flag else efp)[r, g]
            assert Fr(float(reported)) == total, (r, g, float(reported), float(total))
            seq = Fr(0)
            for j in range(16):
                seq = _round_to_f32(errs[j] * errs[j] + seq)
            differs_from_sequential += seq != total
    assert differs_from_sequential > 20


# --------------------------------------------------------------------------- row shards and the random stream

def test_row_shards_with_index_offset_equal_the_whole_tensor(oracle):
    """App. B's random stream runs over the whole tensor.  Quantizing row shards on their own, each with the index
    of its first element as offset and the shared alpha, gives the bytes of the unsharded call."""
    xb = I.generate("cfg4", 48, 256)
    flags = oracle.F_STOCHASTIC | oracle.F_HADAMARD16 | oracle.F_SR_SCALE_17_16
    for fmt in (0, 1, 2, 3, 6):
        c, s, a = oracle.quantize(fmt, xb, flags=flags, sign_mask=0x1234, sr_seed=77)
        parts = [oracle.quantize(fmt, np.ascontiguousarray(xb[lo:hi]), flags=flags | oracle.F_ALPHA_GIVEN, alpha=a,
                                 sign_mask=0x1234, sr_seed=77, sr_index_offset=lo * 256)
                 for lo, hi in ((0, 16), (16, 17), (17, 48))]
        assert np.array_equal(np.concatenate([p[0] for p in parts]), c)
        assert np.array_equal(np.concatenate([p[1] for p in parts]), s)
        wrong = oracle.quantize(fmt, np.ascontiguousarray(xb[16:48]), flags=flags | oracle.F_ALPHA_GIVEN, alpha=a,
                                sign_mask=0x1234, sr_seed=77)
        assert not np.array_equal(wrong[0], c[16:48])                 # without the offset the stream restarts

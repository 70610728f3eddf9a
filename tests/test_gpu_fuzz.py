"""Randomised parity: seeded random shapes, value distributions, formats and options, CUDA path against the
oracle byte for byte (quantize, dequantize, and the transposed entry point where the shape allows)."""
import numpy as np
import pytest

from paper_2603_28765_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    from paper_2603_28765_b200 import binding
    binding.lib()          # raises if the CUDA library is missing: there is no fallback
    return binding


def random_tensor(rng, rows, cols):
    """bf16 bits of one of seven value distributions: normal, heavy-tailed, per-row scales over e^+-9, 90 % zeros,
    small integers times a power of two, a global power-of-two scale up to 2^+-60, 1 % outliers x1000."""
    kind = rng.integers(0, 7)
    if kind == 0:
        x = rng.standard_normal((rows, cols))
    elif kind == 1:
        x = rng.standard_t(2, (rows, cols))
    elif kind == 2:
        x = rng.standard_normal((rows, cols)) * np.exp(rng.normal(0, 3, (rows, 1)))
    elif kind == 3:
        x = rng.standard_normal((rows, cols)) * (rng.random((rows, cols)) < 0.1)
    elif kind == 4:
        x = rng.integers(-8, 9, (rows, cols)).astype(np.float64) * 2.0 ** rng.integers(-20, 20)
    elif kind == 5:
        x = rng.standard_normal((rows, cols)) * 2.0 ** rng.integers(-60, 60)
    else:
        x = rng.standard_normal((rows, cols))
        x[rng.random((rows, cols)) < 0.01] *= 1000
    return I.f32_to_bf16_bits(x.astype(np.float32))


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_cases_match_the_oracle(B, oracle, seed):
    import torch
    rng = np.random.default_rng(seed)
    for case in range(120):
        rows = int(rng.integers(1, 200))
        cols = 16 * int(rng.integers(1, 100))
        xb = random_tensor(rng, rows, cols)
        fmt = int(rng.integers(0, 8))
        flags = 0
        if rng.random() < 0.4:
            flags |= B.ABS_F_HADAMARD16
        if rng.random() < 0.4:
            flags |= B.ABS_F_STOCHASTIC
        if rng.random() < 0.3:
            flags |= B.ABS_F_SR_SCALE_17_16
        mask, sr_seed = int(rng.integers(0, 65536)), int(rng.integers(0, 2 ** 63))
        alpha = None
        if rng.random() < 0.3:
            flags |= B.ABS_F_ALPHA_GIVEN
            amax = float(np.abs(I.bf16_bits_to_f32(xb)).max()) or 1.0
            alpha = float(np.float32(amax / 2688.0 * 2.0 ** rng.integers(-3, 4)))
        where = (seed, case, fmt, flags, rows, cols, alpha)
        x = torch.from_numpy(xb.view(np.int16)).cuda().view(torch.bfloat16)
        ts = torch.tensor([alpha], dtype=torch.float32, device="cuda") if alpha is not None else None
        codes, scales, ts = B.abs_quantize(fmt, x, tensor_scale=ts, opts=B.make_opts(flags, mask, sr_seed))
        out = B.abs_dequantize(fmt, codes, scales, ts, rows, cols)
        torch.cuda.synchronize()
        oc, osc, oa = oracle.quantize(fmt, xb, flags=flags, sign_mask=mask, sr_seed=sr_seed, alpha=alpha)
        assert np.float32(ts.item()).view(np.uint32) == np.float32(oa).view(np.uint32), where
        assert np.array_equal(codes.cpu().numpy()[:oc.size].reshape(oc.shape), oc), where
        assert np.array_equal(scales.cpu().numpy()[:osc.size].reshape(osc.shape), osc), where
        assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16),
                              oracle.dequantize(fmt, oc, osc, oa, rows, cols)), where
        if fmt in (0, 1):                   # the one-pass emulation gives the same dequantized bytes
            od = oracle.dequantize(fmt, oc, osc, oa, rows, cols)
            ts2 = torch.tensor([alpha], dtype=torch.float32, device="cuda") if alpha is not None else None
            eo, _ = B.abs_quantize_dequantize(fmt, x, tensor_scale=ts2, opts=B.make_opts(flags, mask, sr_seed))
            torch.cuda.synchronize()
            assert np.array_equal(eo.view(torch.int16).cpu().numpy().view(np.uint16), od), where
        if fmt in (0, 1) and rows % 16 == 0:
            tf = flags & ~B.ABS_F_ALPHA_GIVEN
            ct, st, at = B.abs_quantize_transposed(fmt, x, opts=B.make_opts(tf, mask, sr_seed))
            torch.cuda.synchronize()
            oc, osc, oa = oracle.quantize(fmt, np.ascontiguousarray(xb.T), flags=tf, sign_mask=mask, sr_seed=sr_seed)
            assert np.float32(at.item()).view(np.uint32) == np.float32(oa).view(np.uint32), where
            assert np.array_equal(ct.cpu().numpy()[:oc.size].reshape(oc.shape), oc), where
            assert np.array_equal(st.cpu().numpy()[:osc.size].reshape(osc.shape), osc), where
            eo, _ = B.abs_quantize_dequantize(fmt, x, opts=B.make_opts(tf | B.ABS_F_GROUPS_DOWN_COLUMNS, mask, sr_seed))
            torch.cuda.synchronize()
            odt = np.ascontiguousarray(oracle.dequantize(fmt, oc, osc, oa, cols, rows).T)
            assert np.array_equal(eo.view(torch.int16).cpu().numpy().view(np.uint16), odt), where

"""abs_quantize_noalloc: the entry point for callers that can no longer allocate device memory
(a server whose own pool already owns all free memory, so cudaMalloc would fail; a loop that cannot
tolerate cudaMalloc's device-wide synchronisation).  Its amax scratch is an array inside the library
image instead of cudaMalloc'ed memory.

The test calls it through the C ABI and requires the same bytes as abs_quantize and as the CPU
reference -- codes, scale bytes and alpha are integer / bit-pattern data, so the comparison is exact,
as everywhere else in this suite -- on calls in a row that share the array (the second tensor has
fewer chunks and a smaller maximum, so anything left over from the first call would show), for every
format, and checks that a call leaves the device's free memory unchanged.  This file sorts last on
purpose: a run that stops at the first failure has then already run every other test.
"""
import ctypes

import numpy as np
import pytest

from paper_2603_28765_b200 import inputs as I

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _dev(xb):
    return torch.from_numpy(xb.view(np.int16)).cuda().view(torch.bfloat16)


def test_noalloc_matches_abs_quantize_on_two_calls_in_a_row(oracle):
    assert torch.cuda.is_available()
    from paper_2603_28765_b200 import binding as B
    L = B.lib()
    first = I.generate("cfg2", 700, 4096)                     # 179200 groups: 22 chunks, ragged last chunk
    second = I.generate("cfg1", 100, 1024, seed=7)             # 6400 groups: one partial chunk, smaller maximum
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    for fmt in sorted(B.FMT_NAMES.values()):                   # every format the entry point dispatches
        for xb in (first, second):
            rows, cols = xb.shape
            x = _dev(xb)
            nb, ns = B.abs_codes_bytes(fmt, rows, cols), B.abs_scales_bytes(fmt, rows, cols)
            want_c, want_s, want_a = B.abs_quantize(fmt, x)
            codes = torch.full((nb,), 0xA5, dtype=torch.uint8, device="cuda")
            scales = torch.full((ns,), 0xA5, dtype=torch.uint8, device="cuda")
            alpha = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
            torch.cuda.synchronize()
            rc = L.abs_quantize_noalloc(fmt, x.data_ptr(), rows, cols, codes.data_ptr(), scales.data_ptr(),
                                        alpha.data_ptr(), stream)
            assert rc == 0, B.status_string(rc)
            torch.cuda.synchronize()
            assert alpha.view(torch.int32).item() == want_a.view(torch.int32).item()
            assert torch.equal(scales, want_s[:ns]) and torch.equal(codes, want_c[:nb])
            # and against the CPU reference directly, not only against the sibling entry point
            oc, osc, oa = oracle.quantize(fmt, xb, threads=8)
            assert np.float32(alpha.item()).view(np.uint32) == np.float32(oa).view(np.uint32)
            assert np.array_equal(codes.cpu().numpy().reshape(rows, -1), oc)
            assert np.array_equal(scales.cpu().numpy().reshape(rows, -1), osc)
            # A further call with everything in place must leave the device's free memory exactly as it was:
            # the entry point allocates nothing, and by now its kernels are loaded.
            free_before, _ = torch.cuda.mem_get_info()
            rc = L.abs_quantize_noalloc(fmt, x.data_ptr(), rows, cols, codes.data_ptr(), scales.data_ptr(),
                                        alpha.data_ptr(), stream)
            assert rc == 0
            torch.cuda.synchronize()
            free_after, _ = torch.cuda.mem_get_info()
            assert free_after == free_before, (fmt, free_before, free_after)
            assert torch.equal(scales, want_s[:ns]) and torch.equal(codes, want_c[:nb])


def test_noalloc_rejects_sizes_beyond_its_static_array():
    from paper_2603_28765_b200 import binding as B
    L = B.lib()
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    codes = torch.zeros(256, dtype=torch.uint8, device="cuda")
    scales = torch.zeros(64, dtype=torch.uint8, device="cuda")
    alpha = torch.zeros(1, dtype=torch.float32, device="cuda")
    too_many_rows = (1 << 30) // 4096 + 1          # one row more than 2**30 elements
    rc = L.abs_quantize_noalloc(B.ABS_FMT_IF4, x.data_ptr(), too_many_rows, 4096, codes.data_ptr(), scales.data_ptr(),
                                alpha.data_ptr(), None)
    assert rc == 7 and "maximum" in B.status_string(rc)     # ABS_ERR_SIZE, nothing enqueued
    assert L.abs_quantize_noalloc(B.ABS_FMT_IF4, x.data_ptr(), 4, 60, codes.data_ptr(), scales.data_ptr(),
                                  alpha.data_ptr(), None) == 2
    torch.cuda.synchronize()

"""hq_conv2d_noalloc - the entry point for callers that may not allocate device memory - against hq_conv2d.

Collected last on purpose: if it fails, a run that stops at the first failure has already run
every other test.  It passes on its own in a fresh process and after the other tests.
"""
from __future__ import annotations

import numpy as np
import pytest

from paper_2011_10680_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

CASES = [
    # n, h, w, cin, cout, k, stride, pad, residual, out_bits: calls in a row on the shared fixed array
    (2, 32, 32, 3, 16, 7, 2, 3, False, 8),
    (1, 20, 20, 5, 32, 3, 1, 1, True, 8),
    (2, 24, 24, 3, 16, 3, 1, 1, False, 4),       # packed 4-bit outputs
    (1, 18, 22, 6, 24, 3, 2, 1, False, 32),      # raw INT32 accumulators
    (4, 228, 228, 3, 64, 7, 2, 3, False, 8),     # patch matrix + weights = 8327680 bytes: just inside the 8 MiB array
]


def test_noalloc_conv_matches_the_allocating_entry_point_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2011_10680_b200 import binding, build
    build.build()
    hq = binding.Handle(0)                      # only for the entry point being compared against
    try:
        for i, (n, h, w, cin, cout, k, stride, pad, residual, out_bits) in enumerate(CASES):
            case = inputs.conv_case(900 + i, n, h, w, cin, cout, k, stride, pad, residual=residual, c_range=(38, 42),
                                    out_bits=out_bits, relu=out_bits != 32)
            dev = binding.upload_case(case)
            st, want = hq.conv_case(case, dev)                     # existing entry point (scratch from cudaMalloc)
            assert st == binding.HQ_OK
            hq.sync()
            got = binding.alloc_out(n, case["ho"], case["wo"], cout, case["out_bits"], case["out_signed"])
            got.fill_(0x5A if got.dtype == torch.uint8 else 0)      # stale bytes must not survive
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            assert binding.conv2d_noalloc(case, dev, got) == binding.HQ_OK
            assert binding.conv2d_noalloc_sync() == binding.HQ_OK   # no bounded device wait ran out
            if i > 0:                                               # the first call loads the library's kernels
                assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
            assert torch.equal(got, want), f"call {i}: results differ from hq_conv2d"   # integers: bit-exact
            from oracle import hqref
            ref = hqref.conv_case(case)
            assert np.array_equal(got.cpu().numpy().view(ref.dtype).reshape(ref.shape), ref)
        # a request beyond the fixed 8 MiB array is refused with a clear status, nothing is launched
        big = inputs.conv_case(990, 4, 230, 230, 3, 64, 7, 2, 3)       # 8474240 bytes: just outside
        dev = binding.upload_case(big)
        out = binding.alloc_out(4, big["ho"], big["wo"], 64, 8, 0)
        assert binding.conv2d_noalloc(big, dev, out) == binding.HQ_ERR_WORKSPACE
        assert binding.status_string(binding.HQ_ERR_WORKSPACE) == "HQ_ERR_WORKSPACE"
    finally:
        hq.close()

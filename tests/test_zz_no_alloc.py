"""ssdq_state_error_static -- the state-error metric for callers that cannot allocate device memory (a server
whose pool owns all of HBM, a hook inside the decode loop) -- gives the numbers of ssdq_state_error.

Collected last on purpose (file name), so that a run stopping at the first failure has already run every
other test.  Called through the C ABI twice in a row: the library-resident scratch keeps the first call's
contents, and the second call, on different data, must not be disturbed by them."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2609_39185_b200 import ssdq

pytestmark = pytest.mark.gpu


def _case(seed, shape, fmt):
    g = torch.Generator(device="cuda").manual_seed(seed)
    B, H, P, N = shape
    twin = torch.randn(shape, generator=g, device="cuda", dtype=torch.float32)
    noisy = twin * (1 + 0.02 * torch.randn(shape, generator=g, device="cuda"))
    if fmt == ssdq.E4M3:
        codes = torch.empty(shape, dtype=torch.uint8, device="cuda")
        scales = torch.empty(B * H * P, dtype=torch.float32, device="cuda")
        ssdq.quantize_store(noisy.view(-1, N), codes.view(-1, N), scales, fmt, ssdq.RTN, 1, scale_block=N)
        return codes, scales, twin, N
    codes = torch.empty(shape, dtype=torch.int16, device="cuda")
    ssdq.quantize_store(noisy.view(-1, N), codes.view(-1, N), None, fmt, ssdq.RTN, 1)
    return codes, None, twin, 0


def test_static_scratch_variant_matches_workspace_variant_twice():
    lib = ssdq.lib()
    stream = torch.cuda.current_stream().cuda_stream
    for seed, shape, fmt in ((1, (6, 40, 8, 128), ssdq.BF16), (2, (3, 7, 64, 64), ssdq.E4M3)):
        codes, scales, twin, sb = _case(seed, shape, fmt)
        B, H, P, N = shape
        want_e, want_r = ssdq.state_error(codes, scales, twin, fmt, sb)
        # the plain float64 definition of the metric, from the CPU oracle
        codes_h = codes.cpu().numpy().view(oracle.CODE_DTYPE[fmt])
        def_e, def_r = oracle.state_error_per_head(codes_h, None if scales is None else scales.cpu().numpy(), twin.cpu().numpy(), fmt, sb)
        got_e = torch.full((H,), -1.0, dtype=torch.float64, device="cuda")
        got_r = torch.full((H,), -1.0, dtype=torch.float64, device="cuda")
        args = (codes.data_ptr(), None if scales is None else scales.data_ptr(), twin.data_ptr(), B, H, P, N, fmt, sb,
                got_e.data_ptr(), got_r.data_ptr(), stream)
        # first call on this device: may load the module and looks up the scratch address
        assert lib.ssdq_state_error_static(*args) == ssdq.OK, lib.ssdq_last_error()
        torch.cuda.synchronize()
        # a later call takes no device memory from anyone: the device-wide free byte count (which, unlike torch's own
        # counters, also sees a cudaMalloc made inside the library) is the same before and after
        got_e.fill_(-1.0)
        got_r.fill_(-1.0)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        assert lib.ssdq_state_error_static(*args) == ssdq.OK, lib.ssdq_last_error()
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        # same kernels and fixed summation order as the workspace variant; the definition to the metric tests' tolerance
        assert np.allclose(got_e.cpu().numpy(), want_e.cpu().numpy(), rtol=1e-10)
        assert np.allclose(got_r.cpu().numpy(), want_r.cpu().numpy(), rtol=1e-10)
        assert np.allclose(got_e.cpu().numpy(), def_e, rtol=1e-10) and np.allclose(got_r.cpu().numpy(), def_r, rtol=1e-10)
        assert float(got_e.min()) > 0.0


def test_static_scratch_variant_rejects_what_does_not_fit():
    lib = ssdq.lib()
    e = torch.zeros(8, dtype=torch.float64, device="cuda")
    big_b, big_h = 1024, 65          # 66560 pairs > 65536
    rc = lib.ssdq_state_error_static(e.data_ptr(), None, e.data_ptr(), big_b, big_h, 1, 16, ssdq.BF16, 0,
                                     e.data_ptr(), e.data_ptr(), None)
    assert rc == ssdq.ERR_SHAPE
    assert b"SSDQ_STATE_ERROR_STATIC_MAX_ITEMS" in lib.ssdq_last_error()

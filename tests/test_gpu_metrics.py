"""GPU sanity-metric kernels against their plain float64 definitions."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39185_b200 import ssdq
from parity import to_dev, codes_to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fmt", [ssdq.FP16, ssdq.BF16, ssdq.E4M3, ssdq.FP32, ssdq.INT8])
def test_state_error_matches_definition(fmt):
    rng = np.random.default_rng(fmt)
    B, H, P, N = 3, 5, 6, 128
    twin = rng.standard_normal((B, H, P, N)).astype(np.float32)
    noisy = (twin * (1 + 0.01 * rng.standard_normal(twin.shape))).astype(np.float32)
    sb = 128 if oracle.has_block_scale(fmt) else 0
    if fmt == ssdq.FP32:
        codes, scales = noisy.view(np.uint32).reshape(-1, N), None
    else:
        codes, scales = oracle.quantize_store(noisy.reshape(-1, N), fmt, oracle.RTN, 1, scale_block=sb)
    codes = codes.reshape(B, H, P, N)
    want_e, want_r = oracle.state_error_per_head(codes, scales, twin, fmt, sb)
    got_e, got_r = ssdq.state_error(codes_to_dev(codes, fmt), to_dev(scales), to_dev(twin), fmt, sb)
    got_e2, got_r2 = ssdq.state_error(codes_to_dev(codes, fmt), to_dev(scales), to_dev(twin), fmt, sb)
    assert np.allclose(got_e.cpu().numpy(), want_e, rtol=1e-10) and np.allclose(got_r.cpu().numpy(), want_r, rtol=1e-10)
    assert torch.equal(got_e, got_e2) and torch.equal(got_r, got_r2)            # fixed summation order


def test_readout_kl_matches_definition():
    rng = np.random.default_rng(9)
    y_ref = (rng.standard_normal((7, 64, 64)) * 3).astype(np.float32)
    y_q = (y_ref + 0.05 * rng.standard_normal(y_ref.shape)).astype(np.float32)
    want = oracle.readout_kl(y_ref, y_q)
    got = ssdq.readout_kl(to_dev(y_ref), to_dev(y_q)).cpu().numpy()
    assert np.allclose(got, want, rtol=1e-5, atol=1e-9)
    assert np.all(ssdq.readout_kl(to_dev(y_ref), to_dev(y_ref)).cpu().numpy() == 0.0)


def test_rule_ordering_on_a_long_horizon():
    """Ordering only (Sections 3 and 6.3): the Weyl dither's state error stays below SR's, and RTN's error
    relative to Weyl's keeps growing with the horizon on an E4M3 store with slow heads."""
    from paper_2609_39185_b200 import sanity, workloads
    cfg = workloads.CONFIGS[4].with_batch(2)
    recs = sanity.run(cfg, 2048, 512, emit=lambda line: None)
    assert [r["step"] for r in recs] == [512, 1024, 1536, 2048]
    for r in recs:
        assert r["weyl"]["state_error"] < r["sr"]["state_error"]
        assert r["weyl"]["readout_kl"] < r["sr"]["readout_kl"]
    ratio = [r["rtn"]["state_error"] / r["weyl"]["state_error"] for r in recs]
    assert ratio[-1] > 1.5 * ratio[0] and ratio[-1] > 1.0

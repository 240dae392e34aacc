"""The bounds-checking build (-DSSDQ_DEBUG): every kernel family runs its parity cases through it with the same bits as
the release build's oracle parity, and no index range it derives leaves the caller's buffers (status word 0).  With
no memory checker available on the GPUs this build is the stand-in: its checks record and skip, they never trap."""
from dataclasses import replace

import numpy as np
import pytest

from paper_2609_39185_b200 import build as ssdq_build
from paper_2609_39185_b200 import ssdq, workloads
from parity import Pair, run_parity

pytestmark = pytest.mark.gpu
CFG = workloads.CONFIGS


@pytest.fixture(scope="module")
def debug_lib():
    ssdq_build.build(debug=True)
    with ssdq.debug_library():
        ssdq.debug_status(reset=True)
        yield
        assert ssdq.debug_status() == (0, 0, 0)


@pytest.mark.parametrize("rule", [ssdq.RTN, ssdq.SR, ssdq.WEYL, ssdq.SR_HASH])
def test_every_kernel_family_stays_inside_its_buffers(debug_lib, rule):
    cases = [(CFG[1], "ssd_update_kernel"),                                                         # tiny, generic kernel
             (replace(CFG[2], batch=3, nheads=200), "ssd_update_mamba1_kernel"),                    # ragged channel tile
             (replace(CFG[5], batch=2, nheads=5, n_layers=1), "ssd_update_tile_kernel"),
             (replace(CFG[4], batch=3, nheads=7), "ssd_update_stream_kernel"),                      # items not a multiple of the grid
             (replace(CFG[4], batch=2, nheads=3, fmt=ssdq.INT8, scale_block=16), "ssd_update_stream_kernel"),
             (replace(CFG[4], batch=2, nheads=3, scale_block=64 * 128), "ssd_update_headscale_kernel"),
             (replace(CFG[3], batch=1, nheads=3, headdim=50), "ssd_update_kernel")]                 # ragged rows per slot
    for cfg, kernel in cases:
        run_parity(cfg, rule, 4, batch_index_base=3)
        assert ssdq.last_kernel() == kernel
        assert ssdq.debug_status() == (0, 0, 0), (cfg.name, kernel)


def test_drivers_and_stand_alone_kernels_run_in_the_debug_build(debug_lib):
    import torch
    cfg = replace(CFG[4], batch=2, nheads=4)
    run_parity(cfg, ssdq.WEYL, 3)
    src = torch.randn(40, 128, device="cuda")
    codes = torch.empty(40, 128, dtype=torch.uint8, device="cuda")
    scales = torch.empty(40, 1, device="cuda")
    ssdq.quantize_store(src, codes, scales, ssdq.E4M3, ssdq.WEYL, 3, weyl=ssdq.weyl_offsets_init(0, 0, 128), scale_block=128)
    torch.cuda.synchronize()
    assert ssdq.debug_status() == (0, 0, 0)

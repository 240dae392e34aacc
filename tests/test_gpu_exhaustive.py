"""Eq. 2 on the local grid, for EVERY finite binary32 input: quantize_store (through the C ABI) against the oracle,
code for code.

The dithered BF16 and FP16 stores run on the hardware stochastic-rounding converts and the E4M3 dither on an
integer form plus a truncating convert, so the rounding of each format is checked on all of its inputs rather than on
samples (Section 2, "Rounding with a threshold": floating-point formats round on the grid spacing of the value's own
binade; Appendix B "Formats").  Thresholds: one value for all entries (0, 2^24 - 1, one mid-range value: a Weyl descriptor whose row and
column multipliers are zero gives every entry the accumulator `base`) and the real Weyl streams at a large write index.

BF16, FP16: all 2^32 - 2^24 finite patterns.  E4M3, INT8: all patterns with |v| <= 448 (127), each block of 16 entries
led by the format's top value so that its scale is exactly 1 and the value reaches the rounding unchanged (what lies
beyond the top cannot occur after scaling).  NaN and infinity are outside the precondition (finite inputs).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39185_b200 import ssdq
from parity import TORCH_CODE, codes_to_host

pytestmark = pytest.mark.gpu

CHUNK = 1 << 26
ROW = 128
CONST_U = [0, (1 << 24) - 1, 0x5A5A5A]
_lane = []


def lane_offsets():
    if not _lane:
        _lane.append(np.arange(CHUNK, dtype=np.uint32))
    return _lane[0]
T_WEYL = 0x80000005


def _const_weyl(U, block):
    """Every entry gets the threshold U: accumulator = base, low 8 bits set to show that they are ignored."""
    w = ssdq.weyl_offsets_init(0, 0, block)
    w.mul_row, w.mul_col, w.base = 0, 0, ((U << 8) | 0xA7) & 0xFFFFFFFF
    return w


def _first_mismatch(got, want, src):
    bad = np.flatnonzero(got.ravel() != want.ravel())
    if len(bad) == 0:
        return None
    i = int(bad[0])
    return (len(bad), hex(int(src.ravel().view(np.uint32)[i])), hex(int(got.ravel()[i])), hex(int(want.ravel()[i])))


@pytest.mark.parametrize("fmt", [ssdq.BF16, ssdq.FP16])
@pytest.mark.parametrize("mode", ["u0", "u1", "weyl"])
def test_every_finite_binary32_through_the_two_byte_dithers(fmt, mode):
    codes = torch.empty((CHUNK // ROW, ROW), dtype=TORCH_CODE[fmt], device="cuda")
    for c in range((1 << 32) // CHUNK):
        bits = lane_offsets() + np.uint32(c * CHUNK)
        if (c & 31) == 31:                                                # the only chunks that hold exponent field 255
            bits[(bits & 0x7F800000) == 0x7F800000] = 0                   # NaN / infinity: not inputs of the method
        src = bits.view(np.float32).reshape(-1, ROW)
        base = c * (CHUNK // ROW)
        if mode == "weyl":
            w = ssdq.weyl_offsets_init(3, 1, 16)
            ssdq.quantize_store(torch.from_numpy(src).cuda(), codes, None, fmt, ssdq.WEYL, T_WEYL, weyl=w, layer=3, row_index_base=base)
            want, _ = oracle.quantize_store(src, fmt, oracle.WEYL, T_WEYL, layer=3, weyl_seed=1, weyl_block=16, row_index_base=base)
        else:
            U = CONST_U[int(mode[1])]
            ssdq.quantize_store(torch.from_numpy(src).cuda(), codes, None, fmt, ssdq.WEYL, 0, weyl=_const_weyl(U, ROW), row_index_base=base)
            want = oracle.round_encode(src, U, fmt, oracle.WEYL)
        torch.cuda.synchronize()
        assert _first_mismatch(codes_to_host(codes, fmt), want, src) is None, (c, _first_mismatch(codes_to_host(codes, fmt), want, src))


@pytest.mark.parametrize("fmt,top,mode", [(ssdq.E4M3, 448.0, "u0"), (ssdq.E4M3, 448.0, "u1"), (ssdq.E4M3, 448.0, "weyl"),
                                          (ssdq.INT8, 127.0, "u1"), (ssdq.INT8, 127.0, "u2"), (ssdq.INT8, 127.0, "weyl"),
                                          (ssdq.INT8, 127.0, "rtn")])
def test_every_binary32_in_range_through_the_one_byte_stores(fmt, top, mode):
    top_bits = int(np.float32(top).view(np.uint32))                       # magnitudes 0 .. top, then the same with the sign bit
    rows = CHUNK // 16
    per_chunk = 15 * rows
    lane = lane_offsets()[:per_chunk]
    codes = torch.empty((rows, 16), dtype=TORCH_CODE[fmt], device="cuda")
    scales = torch.empty((rows, 1), dtype=torch.float32, device="cuda")
    top_code = int(oracle.round_encode(np.float32([top]), None, fmt, oracle.RTN)[0])
    src = np.empty((rows, 16), np.float32)
    src[:, 0] = top
    n_chunks = (top_bits + 1 + per_chunk - 1) // per_chunk
    rule = ssdq.RTN if mode == "rtn" else ssdq.WEYL
    for sign in (0, 0x80000000):
        for c in range(n_chunks):
            bits = np.minimum(lane + np.uint32(c * per_chunk), np.uint32(top_bits)) | np.uint32(sign)    # the tail repeats the top
            src[:, 1:] = bits.view(np.float32).reshape(rows, 15)
            base = (c + (n_chunks if sign else 0)) * rows
            if mode == "weyl":
                w = ssdq.weyl_offsets_init(2, 5, 16)
                ssdq.quantize_store(torch.from_numpy(src).cuda(), codes, scales, fmt, rule, T_WEYL, weyl=w, layer=2, scale_block=16, row_index_base=base)
                want, want_s = oracle.quantize_store(src, fmt, rule, T_WEYL, scale_block=16, layer=2, weyl_seed=5, weyl_block=16, row_index_base=base)
                assert np.all(want_s == 1.0)
            else:
                U = 0 if mode == "rtn" else CONST_U[int(mode[1])]
                ssdq.quantize_store(torch.from_numpy(src).cuda(), codes, scales, fmt, rule, 0, weyl=_const_weyl(U, 16), scale_block=16, row_index_base=base)
                want = oracle.round_encode(src, None if mode == "rtn" else U, fmt, rule)
            torch.cuda.synchronize()
            got = codes_to_host(codes, fmt)
            assert np.all(scales.cpu().numpy() == 1.0)
            assert np.all(got[:, 0] == top_code)                          # the pinning entry itself: floor(top + u) = top
            assert _first_mismatch(got[:, 1:], want[:, 1:], src[:, 1:]) is None, (sign, c, _first_mismatch(got[:, 1:], want[:, 1:], src[:, 1:]))

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

The fixed binary32 routines of Eq. 1 -- the exponential in its scalar and its packed form, and the softplus of the
in-kernel step size -- are compared the same way, on every finite argument, through the fused step itself.
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


def _finite_chunks(chunk):
    """All finite binary32 patterns, `chunk` at a time (NaN and infinity, exponent field 255, replaced by 0)."""
    lane = np.arange(chunk, dtype=np.uint32)
    for c in range((1 << 32) // chunk):
        bits = lane + np.uint32(c * chunk)
        if ((c * chunk) >> 23) & 0xFF == 0xFF or (((c + 1) * chunk - 1) >> 23) & 0xFF == 0xFF:
            bits[(bits & 0x7F800000) == 0x7F800000] = 0
        yield c, bits


def test_every_binary32_argument_of_the_scalar_exponential():
    """exp_spec (Eq. 1's decay a = exp(dt A), evaluated by the fixed binary32 routine) for EVERY finite argument: the
    FP32 twin with one decay per state stores h' = fma(a, 1, 0) = a unrounded, so with h = 1, x = 0 and dt = 1 the state
    after one step is exp_spec(A) entry for entry."""
    H, N = 1 << 22, 16
    f32 = np.float32
    ones = torch.ones((1, H, 1, N), dtype=torch.float32, device="cuda")
    st = torch.empty_like(ones)
    x = torch.zeros((1, H, 1), device="cuda"); dt = torch.ones((1, H), device="cuda")
    Bm = torch.ones((1, N), device="cuda"); Cm = torch.zeros((1, N), device="cuda"); y = torch.empty_like(x)
    A = torch.empty((H, N), dtype=torch.float32, device="cuda")
    desc = ssdq.make_desc(st, None, ssdq.FP32, A=A, D=None, rule=ssdq.RTN)
    for c, bits in _finite_chunks(H * N):
        z = bits.view(f32)
        A.copy_(torch.from_numpy(z.reshape(H, N)))
        st.copy_(ones)
        ssdq.ssd_state_update(desc, 1, x=x, dt=dt, Bm=Bm, Cm=Cm, y=y)
        assert ssdq.last_kernel() == "ssd_update_kernel"
        want = oracle.exp_spec(z)
        got = st.cpu().numpy().reshape(-1)
        assert _first_mismatch(got.view(np.uint32), want.view(np.uint32), z) is None, (c, _first_mismatch(got.view(np.uint32), want.view(np.uint32), z))


def test_every_binary32_argument_of_the_packed_exponential():
    """The Mamba-1 kernel evaluates the same routine on packed pairs (exp_spec2).  Its state is rounded to the store, so
    the decay is read through the readout instead: h = 1, x = 0, dt = 1 and C = the n-th unit vector give y = a[d, n]
    exactly; sixteen launches, one per column, cover the sixteen distinct arguments of every row."""
    H, N = 1 << 22, 16
    f32 = np.float32
    ones = torch.full((1, H, 1, N), 0x3F80, dtype=torch.int16, device="cuda")          # 1.0 in BF16
    st = torch.empty_like(ones)
    x = torch.zeros((1, H, 1), device="cuda"); dt = torch.ones((1, H), device="cuda")
    Bm = torch.ones((1, N), device="cuda"); y = torch.empty_like(x)
    A = torch.empty((H, N), dtype=torch.float32, device="cuda")
    desc = ssdq.make_desc(st, None, ssdq.BF16, A=A, D=None, rule=ssdq.RTN)
    onehot = [torch.zeros((1, N), device="cuda") for _ in range(N)]
    for n in range(N):
        onehot[n][0, n] = 1.0
    got = torch.empty((H, N), dtype=torch.float32, device="cuda")
    for c, bits in _finite_chunks(H * N):
        z = bits.view(f32)
        A.copy_(torch.from_numpy(z.reshape(H, N)))
        for n in range(N):
            st.copy_(ones)
            ssdq.ssd_state_update(desc, 1, x=x, dt=dt, Bm=Bm, Cm=onehot[n], y=y)
            got[:, n] = y.reshape(-1)
        assert ssdq.last_kernel() == "ssd_update_mamba1_kernel"
        want = oracle.exp_spec(z)
        g = got.cpu().numpy().reshape(-1)
        assert _first_mismatch(g.view(np.uint32), want.view(np.uint32), z) is None, (c, _first_mismatch(g.view(np.uint32), want.view(np.uint32), z))


def test_every_binary32_argument_of_the_softplus():
    """softplus_spec (the in-kernel step size dt <- softplus(dt + dt_bias) of a production signature, Appendix B "Runners")
    for EVERY finite argument: with h = 0, A = 0 (a = 1), x = 1, B = 1 the update is h' = fma(1, 0, (dt' * 1) * 1) = dt',
    and C = the first unit vector reads it out as y."""
    H, N = 1 << 22, 16
    f32 = np.float32
    st = torch.zeros((1, H, 1, N), dtype=torch.float32, device="cuda")
    x = torch.ones((1, H, 1), device="cuda"); dt = torch.empty((1, H), device="cuda")
    Bm = torch.ones((1, N), device="cuda"); Cm = torch.zeros((1, N), device="cuda"); y = torch.empty_like(x)
    Cm[0, 0] = 1.0
    A = torch.zeros((H,), dtype=torch.float32, device="cuda")
    desc = ssdq.make_desc(st, None, ssdq.FP32, A=A, D=None, rule=ssdq.RTN, dt_softplus=True)
    for c, bits in _finite_chunks(H):
        z = bits.view(f32)
        dt.copy_(torch.from_numpy(z.reshape(1, H)))
        st.zero_()
        ssdq.ssd_state_update(desc, 1, x=x, dt=dt, Bm=Bm, Cm=Cm, y=y)
        want = oracle.softplus_spec(z)
        got = y.cpu().numpy().reshape(-1)
        assert _first_mismatch(got.view(np.uint32), want.view(np.uint32), z) is None, (c, _first_mismatch(got.view(np.uint32), want.view(np.uint32), z))


@pytest.mark.parametrize("fmt", [ssdq.E4M3, ssdq.INT8, ssdq.INT7, ssdq.INT6, ssdq.INT4])
def test_every_positive_binary32_maximum_through_the_scale_of_the_persistent_kernel(fmt):
    """The persistent one-byte kernel divides the row maximum by the format's constant with a multiply and two fused
    corrections instead of a division.  Every positive finite binary32 maximum: with h = 0, A = 0, dt = 1 and B the first
    unit vector a row's only non-zero entry is h' = x, so its maximum is x and its stored scale must be the oracle's
    max(x / top, FLT_MIN), bit for bit."""
    B, H, P, N = 128, 128, 64, 128
    rows = B * H * P
    st = torch.zeros((B, H, P, N), dtype=torch.uint8, device="cuda")
    sc = torch.ones((rows,), dtype=torch.float32, device="cuda")
    x = torch.empty((B, H, P), device="cuda"); dt = torch.ones((B, H), device="cuda"); y = torch.empty_like(x)
    Bm = torch.zeros((B, N), device="cuda"); Bm[:, 0] = 1.0
    Cm = torch.zeros((B, N), device="cuda")
    A = torch.zeros((H,), device="cuda")
    desc = ssdq.make_desc(st, sc, fmt, A=A, D=None, rule=ssdq.RTN, scale_block=N)
    lane = np.arange(rows, dtype=np.uint32)
    for c in range(0x7F800000 // rows):
        amax = (lane + np.uint32(c * rows)).view(np.float32)
        x.copy_(torch.from_numpy(amax.reshape(B, H, P)))
        st.zero_()
        ssdq.ssd_state_update(desc, 1, x=x, dt=dt, Bm=Bm, Cm=Cm, y=y)
        assert ssdq.last_kernel() == "ssd_update_stream_kernel"
        want = oracle.block_scale(amax, fmt)
        got = sc.cpu().numpy()
        assert _first_mismatch(got.view(np.uint32), want.view(np.uint32), amax) is None, (c, _first_mismatch(got.view(np.uint32), want.view(np.uint32), amax))

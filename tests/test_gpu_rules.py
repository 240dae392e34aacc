"""GPU parity of the rule machinery in isolation (through the C ABI): thresholds and quantize_store
against the CPU oracle, bit for bit."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2609_39185_b200 import ssdq
from parity import to_dev, codes_to_host, TORCH_CODE

pytestmark = pytest.mark.gpu

FMTS = [ssdq.FP16, ssdq.BF16, ssdq.E4M3]
INT_FMTS = [ssdq.INT8, ssdq.INT7, ssdq.INT6, ssdq.INT4]
RULES = [ssdq.RTN, ssdq.SR, ssdq.WEYL, ssdq.SR_HASH]


@pytest.mark.parametrize("first_flat", [0, 12345, 2**32 - 100, 2**36 + 3])
@pytest.mark.parametrize("block", [16, 128])
def test_weyl_thresholds_match_oracle(first_flat, block):
    n = 5000
    for layer, seed, t in ((0, 0, 1), (5, 1, 4096), (7, 3, 2**32 - 1)):
        w = ssdq.weyl_offsets_init(layer, seed, block)
        got = ssdq.thresholds_materialize(ssdq.WEYL, n, t, weyl=w, first_flat=first_flat).cpu().numpy().view(np.uint32)
        want = oracle.thresholds(oracle.WEYL, range(first_flat, first_flat + n), t, layer=layer, weyl_seed=seed, weyl_block=block)
        assert np.array_equal(got, want)


@pytest.mark.parametrize("first_flat", [0, 7, 2**34 + 1, 2**32 - 50])
@pytest.mark.parametrize("rule", [ssdq.SR, ssdq.SR_HASH])
def test_sr_thresholds_match_oracle(first_flat, rule):
    n = 4099
    for layer, seed, t in ((0, 0, 1), (3, 0xDEADBEEFCAFE, 77)):
        got = ssdq.thresholds_materialize(rule, n, t, sr_seed=seed, layer=layer, first_flat=first_flat).cpu().numpy().view(np.uint32)
        want = oracle.thresholds(rule, range(first_flat, first_flat + n), t, layer=layer, sr_seed=seed)
        assert np.array_equal(got, want)


def value_zoo(rng, n_rows, row_len, fmt):
    """float32 rows that exercise every branch of Eq. 2 on the local grid: all binades of the format
    including its subnormal range and values below it, exact grid points, zeros of both signs,
    values beyond the largest finite number."""
    lo, hi = {ssdq.FP16: (-50, 17), ssdq.BF16: (-126, 127), ssdq.E4M3: (-40, 10)}.get(fmt, (-40, 10))
    n = n_rows * row_len
    e = rng.integers(lo, hi + 1, n)
    m = rng.integers(0, 1 << 23, n).astype(np.uint32)
    keep = {ssdq.FP16: 10, ssdq.BF16: 7, ssdq.E4M3: 3}.get(fmt, 6)
    m[::5] &= np.uint32(~((1 << (23 - keep)) - 1) & 0x7FFFFF)      # exact grid points (in the normal range)
    m[1::11] = 0x7FFFFF                                             # just below a binade boundary
    s = rng.integers(0, 2, n).astype(np.uint32)
    bits = (s << 31) | ((e + 127).astype(np.uint32) << 23) | m
    bits[2::97] = 0
    bits[3::97] = 0x80000000
    bits[4::97] = rng.integers(1, 1 << 23, len(bits[4::97])).astype(np.uint32)          # binary32 subnormals
    bits[5::97] = 0x80000000 | rng.integers(1, 1 << 23, len(bits[5::97])).astype(np.uint32)
    return bits.view(np.float32).reshape(n_rows, row_len)


@pytest.mark.parametrize("fmt", FMTS + INT_FMTS)
@pytest.mark.parametrize("rule", RULES)
@pytest.mark.parametrize("row_len,weyl_block,scale_block", [(128, 128, 128), (128, 16, 16), (16, 16, 16), (64, 16, 64), (256, 16, 16), (32, 16, 32)])
def test_quantize_store_matches_oracle(fmt, rule, row_len, weyl_block, scale_block):
    rng = np.random.default_rng(1000 * fmt + 10 * rule + row_len)
    n_rows = 700                                                    # not a multiple of the slots per CTA
    src = value_zoo(rng, n_rows, row_len, fmt)
    sb = scale_block if oracle.has_block_scale(fmt) else 0
    if fmt in INT_FMTS:      # integer grids: mix blocks of ordinary magnitudes with the zoo (whose blocks are dominated by one huge entry)
        src[::2] = (rng.standard_normal((len(src[::2]), row_len)) * rng.uniform(1e-3, 50, (len(src[::2]), 1))).astype(np.float32)
    base, t, layer, seed = 2**30 + 5, 1234567, 4, 99
    want_codes, want_scales = oracle.quantize_store(src, fmt, rule, t, scale_block=sb, layer=layer, weyl_seed=1,
                                                    weyl_block=weyl_block, sr_seed=seed, row_index_base=base)
    codes = torch.zeros((n_rows, row_len), dtype=TORCH_CODE[fmt], device="cuda")
    scales = torch.zeros((n_rows, row_len // sb), dtype=torch.float32, device="cuda") if sb else None
    w = ssdq.weyl_offsets_init(layer, 1, weyl_block)
    ssdq.quantize_store(to_dev(src), codes, scales, fmt, rule, t, weyl=w, sr_seed=seed, layer=layer, scale_block=sb,
                        row_index_base=base)
    torch.cuda.synchronize()
    got = codes_to_host(codes, fmt)
    bad = np.argwhere(got != want_codes)
    assert len(bad) == 0, (len(bad), src[tuple(bad[0])].item().hex(), hex(int(got[tuple(bad[0])])), hex(int(want_codes[tuple(bad[0])])))
    if sb:
        assert np.array_equal(scales.cpu().numpy().view(np.uint32), want_scales.view(np.uint32))


@pytest.mark.parametrize("fmt", [ssdq.FP16, ssdq.E4M3])
def test_subnormal_decision_boundary(fmt):
    """Values below the format's normal range whose kept bits sit exactly on the round-up boundary:
    the dropped low bits of the value and of the threshold decide.  Thresholds are steered by solving
    the Weyl accumulator for the write index t (Phi is odd, hence invertible modulo 2^32)."""
    mant, emin = {ssdq.FP16: (10, -14), ssdq.E4M3: (3, -6)}[fmt]
    drop = 23 - mant
    phi_inv = pow(2654435769, -1, 2**32)
    w = ssdq.weyl_offsets_init(0, 0, 16)
    rng = np.random.default_rng(7 + fmt)
    row_len, n_rows = 16, 64
    for trial in range(24):
        # one write index t per trial; entry (0, 0) is steered onto the boundary, the rest is a zoo
        e = int(rng.integers(emin - 30, emin))                     # subnormal target
        mbits = int(rng.integers(0, 1 << 23))
        sign = int(rng.integers(0, 2))
        v = np.uint32((sign << 31) | ((e + 127) << 23) | mbits).view(np.float32)
        # kept fraction bits F of |v| on the first binade: mantissa of |v| + 2^emin, truncated
        F = int(Fraction(abs(float(v))) / Fraction(2) ** (emin - 23)) & ((1 << drop) - 1)
        r_needed = ((1 << drop) - 1) - F                           # F + r == all ones
        low = int(rng.integers(0, 1 << (32 - drop)))
        acc_top = r_needed if sign == 0 else ((1 << drop) - 1) - r_needed
        target_acc = ((acc_top << (32 - drop)) | low) & 0xFFFFFFFF
        # acc(r=0, c=0, t) = mul_row + mul_col + base + t*phi  =>  t
        t = ((target_acc - (w.mul_row + w.mul_col + w.base)) * phi_inv) % 2**32
        src = value_zoo(rng, n_rows, row_len, fmt)
        src[0, 0] = v
        sb = 16 if fmt == ssdq.E4M3 else 0
        if fmt == ssdq.E4M3:
            src[0, 1:] = 0.0
            src[0, 1] = 448.0          # block scale exactly 1: the steered value reaches the rounding unchanged
        want_codes, _ = oracle.quantize_store(src, fmt, ssdq.WEYL, t, scale_block=sb, weyl_block=16)
        codes = torch.zeros((n_rows, row_len), dtype=TORCH_CODE[fmt], device="cuda")
        scales = torch.zeros((n_rows, 1), dtype=torch.float32, device="cuda") if sb else None
        ssdq.quantize_store(to_dev(src), codes, scales, fmt, ssdq.WEYL, t, weyl=w, scale_block=sb)
        torch.cuda.synchronize()
        assert np.array_equal(codes_to_host(codes, fmt), want_codes), trial


@pytest.mark.parametrize("fmt", FMTS + [ssdq.FP32, ssdq.INT8, ssdq.INT4])
def test_dequantize_matches_oracle(fmt):
    rng = np.random.default_rng(3)
    n_rows, row_len = 33, 128
    sb = 128 if oracle.has_block_scale(fmt) else 0
    if fmt == ssdq.FP32:
        codes_h = rng.standard_normal((n_rows, row_len)).astype(np.float32).view(np.uint32)
        scales_h = None
    else:
        codes_h, scales_h = oracle.quantize_store(rng.standard_normal((n_rows, row_len)).astype(np.float32) * 3, fmt,
                                                  oracle.RTN, 1, scale_block=sb)
    from parity import codes_to_dev
    out = torch.empty((n_rows, row_len), dtype=torch.float32, device="cuda")
    ssdq.dequantize(codes_to_dev(codes_h, fmt), to_dev(scales_h), fmt, out, scale_block=sb)
    want = oracle.dequantize(codes_h, scales_h, fmt, sb)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_exp_and_softplus_kernels_reproduce_the_known_answer_table(golden_dir):
    """The frozen table guards both sides against a silent, matching change.  exp_spec: FP32-twin state h = 1, x = 0,
    dt = 1, A = z, so the stored h' is a = exp_spec(z).  softplus_spec: h = 0, A = 0, x = B = 1 and in-kernel softplus,
    so the stored h' is the step size softplus_spec(dt_raw)."""
    from test_oracle_update import load_spec_kat
    kat = load_spec_kat(golden_dir)
    N = 16
    for name in ("exp_spec", "softplus_spec"):
        zin, zout = kat[name]
        H = len(zin)
        z = torch.from_numpy(zin.view(np.float32).copy()).cuda()
        one = torch.ones((1, H), dtype=torch.float32, device="cuda")
        y = torch.empty((1, H, 1), dtype=torch.float32, device="cuda")
        if name == "exp_spec":
            state = torch.ones((1, H, 1, N), dtype=torch.float32, device="cuda")
            d = ssdq.make_desc(state, None, ssdq.FP32, A=z, D=None, rule=ssdq.RTN)
            ssdq.ssd_state_update(d, 1, x=torch.zeros((1, H, 1), device="cuda"), dt=one, Bm=torch.ones((1, N), device="cuda"),
                                  Cm=torch.zeros((1, N), device="cuda"), y=y)
        else:
            state = torch.zeros((1, H, 1, N), dtype=torch.float32, device="cuda")
            d = ssdq.make_desc(state, None, ssdq.FP32, A=torch.zeros(H, device="cuda"), D=None, rule=ssdq.RTN, dt_softplus=True)
            ssdq.ssd_state_update(d, 1, x=torch.ones((1, H, 1), device="cuda"), dt=z.view(1, H), Bm=torch.ones((1, N), device="cuda"),
                                  Cm=torch.zeros((1, N), device="cuda"), y=y)
        torch.cuda.synchronize()
        got = state.cpu().numpy().view(np.uint32)[0, :, 0, :]
        assert np.array_equal(got, np.repeat(zout[:, None], N, axis=1)), name


def _contraction_sensitive_tie():
    """(amax, h, k_even): the block scale s = amax / 127 and h are such that RN(h * RN(1/s)) is exactly k + 1/2 while the
    exact product is not: a multiply that is fused into the rounding add would round to the nearer integer instead of
    the even one.  Checked here in exact arithmetic before it is used."""
    f32 = np.float32
    s = np.uint32(1021728416).view(f32)
    h = np.uint32(3196633967).view(f32)
    amax = None
    for cand in np.nextafter(f32(s * f32(127.0)), [f32(0), f32(1e9)], dtype=f32).tolist() + [float(f32(s * f32(127.0)))]:
        if f32(f32(cand) / f32(127.0)) == s:
            amax = f32(cand)
    assert amax is not None
    rinv = f32(f32(1.0) / s)
    v = f32(h * rinv)
    exact = Fraction(float(h)) * Fraction(float(rinv))
    assert float(v) == -9.5 and exact != Fraction(-19, 2) and exact > Fraction(-19, 2)      # nearest of the exact product: -9; ties-to-even of v: -10
    return amax, h, -10


def test_int8_rtn_tie_is_not_moved_by_a_fused_multiply_add():
    """v = h' * (1/s) is rounded BEFORE it is rounded onto the integer grid (two operations); every kernel that writes
    INT8 codes must keep the tie: quantize_store, the persistent kernel, the per-head-scale kernel and the generic one."""
    amax, h, want = _contraction_sensitive_tie()
    N = 128
    row = np.zeros(N, np.float32)
    row[0], row[1], row[17] = amax, h, h
    want_row = oracle.quantize_store(row.reshape(1, N), oracle.INT8, oracle.RTN, 1, scale_block=N)[0].view(np.int8)[0]
    assert want_row[1] == want and want_row[17] == want and want_row[0] == 127
    # quantize_store
    src = np.tile(row, (64, 1))
    codes = torch.zeros((64, N), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((64, 1), dtype=torch.float32, device="cuda")
    ssdq.quantize_store(to_dev(src), codes, scales, ssdq.INT8, ssdq.RTN, 1, scale_block=N)
    assert np.array_equal(codes.cpu().numpy().view(np.int8), np.tile(want_row, (64, 1)))
    # the decode step: zero state, A = 0 (a = 1), dt = x = 1, so h' = B[n] on every row
    for shape, sb, kernel in (((2, 3, 64, N), N, "ssd_update_stream_kernel"), ((2, 3, 64, N), 64 * N, "ssd_update_headscale_kernel"),
                              ((2, 3, 5, N), N, "ssd_update_kernel"), ((2, 3, 32, N), N, "ssd_update_tile_kernel")):
        B, H, P, _ = shape
        state = torch.zeros(shape, dtype=torch.uint8, device="cuda")
        sc = torch.full((B * H * P * N // sb,), float(np.finfo(np.float32).tiny), dtype=torch.float32, device="cuda")
        d = ssdq.make_desc(state, sc, ssdq.INT8, A=torch.zeros(H, device="cuda"), D=None, rule=ssdq.RTN, scale_block=sb)
        ssdq.ssd_state_update(d, 1, x=torch.ones((B, H, P), device="cuda"), dt=torch.ones((B, H), device="cuda"),
                              Bm=to_dev(np.tile(row, (B, 1))), Cm=torch.zeros((B, N), device="cuda"),
                              y=torch.empty((B, H, P), device="cuda"))
        torch.cuda.synchronize()
        assert ssdq.last_kernel() == kernel
        got = state.cpu().numpy().view(np.int8).reshape(-1, N)
        assert np.array_equal(got, np.tile(want_row, (len(got), 1))), kernel

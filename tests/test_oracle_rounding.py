"""Pins of the oracle's formats and of Eq. 2 on the local grid.

The reference grid of each format is enumerated from torch's CPU view-casts of every storage code
(an independent statement of the formats); Eq. 2 is then checked in its case form -- round up to the
next grid point iff u >= 1 - f -- with f computed in exact rational arithmetic."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import FP16, BF16, E4M3, RTN, SR, WEYL, SR_HASH

TORCH_DTYPE = {FP16: torch.float16, BF16: torch.bfloat16, E4M3: torch.float8_e4m3fn}
MAX_FINITE = {FP16: 65504.0, BF16: float(np.float32(3.3895313892515355e38)), E4M3: 448.0}


def all_codes(fmt):
    if fmt == E4M3:
        return np.arange(256, dtype=np.uint8)
    return np.arange(65536, dtype=np.int64).astype(np.uint16)


def torch_decode(codes, fmt):
    if fmt == E4M3:
        t = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn)
    else:
        t = torch.from_numpy(codes.view(np.int16).copy()).view(TORCH_DTYPE[fmt])
    return t.to(torch.float32).numpy()


def grid_of(fmt):
    vals = torch_decode(all_codes(fmt), fmt).astype(np.float64)
    vals = vals[np.isfinite(vals)]
    return np.unique(vals)          # sorted; -0 and +0 merge


@pytest.mark.parametrize("fmt", [FP16, BF16, E4M3])
def test_decode_and_encode_match_library_view_casts(fmt):
    codes = all_codes(fmt)
    want = torch_decode(codes, fmt)
    got = oracle.decode(codes, fmt)
    finite = np.isfinite(want)
    assert np.array_equal(np.isnan(want), np.isnan(got))
    assert np.array_equal(want[~np.isnan(want)].view(np.uint32), got[~np.isnan(got)].view(np.uint32))
    back = oracle.encode(want[finite], fmt)
    assert np.array_equal(back, codes[finite])           # includes -0 -> sign bit only


def sample_values(rng, n, lo_exp, hi_exp):
    """Random float32 values spread over binades [2^lo_exp, 2^hi_exp), both signs."""
    e = rng.integers(lo_exp, hi_exp, n)
    m = rng.integers(0, 1 << 23, n).astype(np.uint32)
    s = rng.integers(0, 2, n).astype(np.uint32)
    bits = (s << 31) | ((e + 127).astype(np.uint32) << 23) | m
    return bits.view(np.float32)


@pytest.mark.parametrize("fmt,lo,hi", [(FP16, -27, 16), (BF16, -60, 60), (E4M3, -12, 9)])
def test_rtn_matches_native_casts_bit_for_bit(fmt, lo, hi):
    # Appendix B "Formats": round-to-nearest matches native casts bit for bit on 2e5 values over 34+ binades
    rng = np.random.default_rng(fmt)
    v = sample_values(rng, 200000, lo, hi)
    ties = torch_decode(all_codes(fmt), fmt)
    ties = ties[np.isfinite(ties)]
    mid = ((ties[:-1].astype(np.float64) + np.roll(ties, -1)[:-1].astype(np.float64)) / 2).astype(np.float32)
    v = np.concatenate([v, mid[np.isfinite(mid)], ties])
    v = v[np.abs(v) <= MAX_FINITE[fmt]]                      # saturation is pinned separately
    want = torch.from_numpy(v).to(TORCH_DTYPE[fmt]).to(torch.float32).numpy()
    got = oracle.round_values(v, 0, fmt, RTN)
    assert np.array_equal(want.view(np.uint32), got.view(np.uint32))


def expected_eq2(v, U, grid, max_finite):
    """Eq. 2, case form, on an enumerated grid: lo <= v <= hi neighbours, f = (v - lo)/(hi - lo)."""
    if abs(v) > max_finite:
        return float(np.copysign(max_finite, v)), None
    i = int(np.searchsorted(grid, v, side="right")) - 1
    lo = grid[i]
    if lo == v:
        return float(v), Fraction(0)
    hi = grid[i + 1]
    f = (Fraction(float(v)) - Fraction(float(lo))) / (Fraction(float(hi)) - Fraction(float(lo)))
    up = Fraction(U, 1 << 24) >= 1 - f
    return float(hi if up else lo), f


@pytest.mark.parametrize("fmt,lo,hi", [(FP16, -40, 17), (BF16, -140, 128), (E4M3, -30, 10)])
def test_dithered_rounding_is_eq2_on_the_enumerated_grid(fmt, lo, hi):
    rng = np.random.default_rng(10 + fmt)
    grid = grid_of(fmt)
    n = 6000
    v = sample_values(rng, n, max(lo, -126), min(hi, 127))
    if fmt == BF16:   # binary32 subnormals are BF16 subnormal targets
        sub = (rng.integers(1, 1 << 23, 500).astype(np.uint32) | (rng.integers(0, 2, 500).astype(np.uint32) << 31))
        v = np.concatenate([v, sub.view(np.float32)])
    U = rng.integers(0, 1 << 24, len(v)).astype(np.uint32)
    U[::7] = 0
    U[1::7] = (1 << 24) - 1
    U[2::7] = 1
    U[3::7] = 1 << 23
    got = oracle.round_values(v, U, fmt, WEYL)
    assert np.array_equal(got.view(np.uint32), oracle.round_values(v, U, fmt, SR).view(np.uint32))
    for vi, Ui, gi in zip(v, U, got):
        want, _ = expected_eq2(float(vi), int(Ui), grid, MAX_FINITE[fmt])
        assert float(gi) == want, (float(vi).hex(), int(Ui), float(gi), want)
        if gi == 0.0:
            assert np.signbit(gi) == np.signbit(vi)          # a value rounded to zero keeps its sign


@pytest.mark.parametrize("fmt", [FP16, BF16, E4M3])
def test_round_up_probability_is_exactly_f(fmt):
    # SR "rounds up with probability exactly f": the number of 24-bit thresholds that round up is
    # f * 2^24 rounded down to an integer, and the switch sits exactly at U* = ceil((1 - f) * 2^24).
    rng = np.random.default_rng(20 + fmt)
    grid = grid_of(fmt)
    lo_e, hi_e = {FP16: (-26, 15), BF16: (-100, 100), E4M3: (-11, 8)}[fmt]
    for vi in sample_values(rng, 300, lo_e, hi_e):
        _, f = expected_eq2(float(vi), 0, grid, MAX_FINITE[fmt])
        if f is None or f == 0:
            continue
        ustar = -((-(1 - f) * (1 << 24)) // 1)           # ceil
        ustar = int(ustar)
        below = oracle.round_values(vi, max(ustar - 1, 0), fmt, WEYL)[0]
        down = expected_eq2(float(vi), 0, grid, MAX_FINITE[fmt])[0]
        assert float(below) == down
        if ustar < (1 << 24):
            above = oracle.round_values(vi, ustar, fmt, WEYL)[0]
            assert float(above) > down if vi > 0 or down != 0 else True
            assert float(above) != float(below)


def test_tiny_values_and_signed_floor():
    # Eq. 2 is a floor of the signed value: a tiny positive value never rounds up, a tiny negative
    # value reaches -step only for u = 0; the stored zero keeps the sign.
    tiny = np.float32(1e-30)
    step16 = 2.0**-24
    assert oracle.round_values(tiny, (1 << 24) - 1, FP16, WEYL)[0] == 0.0
    assert oracle.round_values(-tiny, 0, FP16, WEYL)[0] == -step16
    r = oracle.round_values(-tiny, 1, FP16, WEYL)[0]
    assert r == 0.0 and np.signbit(r)
    # a negative value moves towards +inf with probability equal to its signed fraction
    v = np.float32(-(1.0 + 0.25 * 2.0**-10))                 # -(1 + s/4) on the fp16 grid near 1
    ups = sum(float(oracle.round_values(v, U, FP16, WEYL)[0]) == -1.0 for U in range(0, 1 << 24, 1 << 12))
    assert ups == 3 * (1 << 12) // 4


@pytest.mark.parametrize("fmt", [FP16, BF16, E4M3])
def test_saturation_and_rtn_ties(fmt):
    big = np.float32(MAX_FINITE[fmt]) * np.float32(1.5) if fmt != BF16 else np.float32(3.4e38)
    for rule, U in ((RTN, 0), (WEYL, 0), (WEYL, (1 << 24) - 1)):
        assert oracle.round_values(big, U, fmt, rule)[0] == np.float32(MAX_FINITE[fmt])
        assert oracle.round_values(-big, U, fmt, rule)[0] == -np.float32(MAX_FINITE[fmt])
    # E4M3: between 448 and the (unrepresentable) next step 480 everything saturates to 448
    if fmt == E4M3:
        assert oracle.round_values(np.float32(470.0), (1 << 24) - 1, E4M3, WEYL)[0] == 448.0
        assert oracle.round_values(np.float32(470.0), 0, E4M3, RTN)[0] == 448.0
    # ties go to even under RTN (native-cast semantics), not up
    if fmt == FP16:
        s = 2.0**-10
        assert oracle.round_values(np.float32(1.0 + 0.5 * s), 0, FP16, RTN)[0] == 1.0
        assert oracle.round_values(np.float32(1.0 + 1.5 * s), 0, FP16, RTN)[0] == np.float32(1.0 + 2 * s)


@pytest.mark.parametrize("rule", [SR, WEYL, SR_HASH])
def test_dithers_are_unbiased_and_lemma_2_noise(rule):
    # E[Q_u(x)] = x over a long run (Section 2), and Lemma 2: with f uniform the mean squared
    # residual is s^2/12 under RTN and s^2/6 under SR or the Weyl dither.
    s = 2.0**-10                                               # fp16 spacing in [1, 2)
    T = 4096
    x = np.float32(1.0 + 0.3 * s)
    U = np.array([oracle.threshold(rule, flat=5, t=t, weyl_block=16) for t in range(1, T + 1)], dtype=np.uint32)
    q = oracle.round_values(np.full(T, x, dtype=np.float32), U, FP16, rule).astype(np.float64)
    tol = 4 * s / T if rule == WEYL else 4 * s * np.sqrt(0.3 * 0.7 / T)
    assert abs(q.mean() - float(x)) < tol
    rng = np.random.default_rng(3)
    n = 200000
    xs = (1.0 + rng.random(n)).astype(np.float32)             # f uniform, independent of the threshold
    U = np.array([oracle.threshold(rule, flat=int(i), t=7, weyl_block=16) for i in range(n)], dtype=np.uint32)
    res = (oracle.round_values(xs, U, FP16, rule).astype(np.float64) - xs.astype(np.float64)) / s
    assert abs(np.mean(res**2) - 1 / 6) < 0.004
    res = (oracle.round_values(xs, 0, FP16, RTN).astype(np.float64) - xs.astype(np.float64)) / s
    assert abs(np.mean(res**2) - 1 / 12) < 0.002


@pytest.mark.parametrize("fmt,lo,hi", [(FP16, -60, 18), (BF16, -126, 127), (E4M3, -40, 10)])
def test_dithered_rounding_on_a_million_values(fmt, lo, hi):
    """The case form of Eq. 2 on the enumerated grid, vectorised in float64 (every quantity below is exact in
    float64: grid points and values are binary32 numbers, the spacing is a power of two, u is a multiple of 2^-24)."""
    rng = np.random.default_rng(30 + fmt)
    grid = grid_of(fmt)
    n = 1_000_000
    v = sample_values(rng, n, lo, hi)
    v[::1000] = 0.0
    v = v[np.abs(v) <= MAX_FINITE[fmt]]
    U = rng.integers(0, 1 << 24, len(v)).astype(np.uint32)
    U[::9] = 0
    U[1::9] = (1 << 24) - 1
    vd = v.astype(np.float64)
    i = np.searchsorted(grid, vd, side="right") - 1
    lo_pt = grid[i]
    hi_pt = grid[np.minimum(i + 1, len(grid) - 1)]
    on_grid = lo_pt == vd
    step = np.where(on_grid, 1.0, hi_pt - lo_pt)
    f = (vd - lo_pt) / step
    up = (U.astype(np.float64) / 2.0**24 >= 1.0 - f) & ~on_grid
    want = np.where(up, hi_pt, lo_pt)
    got = oracle.round_values(v, U, fmt, WEYL).astype(np.float64)
    assert np.array_equal(got, want)
    zero = got == 0.0
    assert np.array_equal(np.signbit(got[zero]), np.signbit(v[zero]))


@pytest.mark.parametrize("fmt", [FP16, BF16, E4M3])
def test_rtn_matches_native_casts_on_two_million_values(fmt):
    rng = np.random.default_rng(40 + fmt)
    lo, hi = {FP16: (-60, 16), BF16: (-126, 127), E4M3: (-40, 9)}[fmt]
    v = sample_values(rng, 2_000_000, lo, hi)
    v = v[np.abs(v) <= MAX_FINITE[fmt]]
    want = torch.from_numpy(v).to(TORCH_DTYPE[fmt]).to(torch.float32).numpy()
    got = oracle.round_values(v, 0, fmt, RTN)
    assert np.array_equal(want.view(np.uint32), got.view(np.uint32))

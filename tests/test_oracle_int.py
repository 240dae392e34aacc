"""Pins of the oracle's symmetric block-absmax integer stores (Appendix B "Formats", INTb): uniform grid,
q_max = 2^(b-1) - 1, FP32 block scale max|h| / q_max, clamp to [-q_max, q_max]."""
from fractions import Fraction
import math

import numpy as np
import pytest

import oracle
from oracle import INT8, INT7, INT6, INT4, RTN, SR, WEYL, INT_QMAX

INTS = [INT8, INT7, INT6, INT4]


@pytest.mark.parametrize("fmt", INTS)
def test_rtn_is_rint_with_clamp(fmt):
    q = INT_QMAX[fmt]
    rng = np.random.default_rng(fmt)
    v = np.concatenate([rng.uniform(-q - 3, q + 3, 20000), np.arange(-q - 2, q + 2) + 0.5,
                        np.arange(-q - 2, q + 3, dtype=np.float64), [1e-30, -1e-30, 0.0, -0.0, 1e30, -1e30]]).astype(np.float32)
    got = oracle.round_values(v, 0, fmt, RTN)
    want = np.clip(np.rint(v.astype(np.float64)), -q, q)              # numpy rint: ties to even
    assert np.array_equal(got.astype(np.float64), want)
    codes = oracle.encode(got, fmt).view(np.int8)
    assert np.array_equal(codes.astype(np.float64), want)
    assert np.array_equal(oracle.decode(codes.view(np.uint8), fmt).astype(np.float64), want)


@pytest.mark.parametrize("fmt", INTS)
def test_dither_is_eq2_on_the_integer_grid(fmt):
    q = INT_QMAX[fmt]
    rng = np.random.default_rng(10 + fmt)
    v = np.concatenate([rng.uniform(-q - 2, q + 2, 4000), rng.uniform(-1, 1, 500) * 1e-6]).astype(np.float32)
    U = rng.integers(0, 1 << 24, len(v)).astype(np.uint32)
    U[::5] = 0
    U[1::5] = (1 << 24) - 1
    got = oracle.round_values(v, U, fmt, WEYL)
    for vi, Ui, gi in zip(v, U, got):
        x = Fraction(float(vi))
        k = math.floor(x)
        f = x - k
        want = k + (1 if Fraction(int(Ui), 1 << 24) >= 1 - f else 0)       # Eq. 2, case form (f = 0: never up)
        if f == 0:
            want = k
        assert float(gi) == float(min(max(want, -q), q))


@pytest.mark.parametrize("fmt", INTS)
@pytest.mark.parametrize("block", [16, 128])
def test_block_scale_and_no_clipping_with_an_fp32_scale(fmt, block):
    q = INT_QMAX[fmt]
    rng = np.random.default_rng(20 + fmt)
    src = (rng.standard_normal((64, 128)) * rng.uniform(1e-3, 10, (64, 1))).astype(np.float32)
    src[3] = 0.0
    codes, scales = oracle.quantize_store(src, fmt, RTN, 1, scale_block=block)
    blocks = src.reshape(64, 128 // block, block)
    amax = np.abs(blocks).max(axis=2)
    want_s = np.maximum((amax / np.float32(q)).astype(np.float32), np.finfo(np.float32).tiny)
    assert np.array_equal(scales, want_s)
    k = codes.view(np.int8).reshape(blocks.shape).astype(np.int32)
    assert np.abs(k).max() <= q
    nz = amax > 0
    assert np.all(np.abs(k).max(axis=2)[nz] == q)                       # the block maximum lands on q_max: not clipped
    deq = oracle.dequantize(codes, scales, fmt, block).reshape(blocks.shape)
    assert np.all(np.abs(deq - blocks) <= 0.5 * scales[..., None] * (1 + 1e-5))
    for rule in (SR, WEYL):
        c2, s2 = oracle.quantize_store(src, fmt, rule, 5, scale_block=block, weyl_block=16)
        d2 = oracle.dequantize(c2, s2, fmt, block).reshape(blocks.shape)
        assert np.array_equal(s2, scales)
        assert np.all(np.abs(d2 - blocks) <= scales[..., None] * (1 + 1e-5))
        assert np.abs(c2.view(np.int8).astype(np.int32)).max() <= q


def int_recurrence(fmt, fracs, h0, T, rule):
    """A block of 16 entries whose scale is pinned to exactly 1: entry 0 holds q_max with a = 1 and no write,
    the other 15 accumulate a constant write w = m + f per step (a = 1, dt = x = 1, B[n] = w[n])."""
    q = INT_QMAX[fmt]
    N = 16
    st = np.zeros((1, 1, 1, N), np.uint8)
    st[0, 0, 0, 0] = q
    st[0, 0, 0, 1:] = np.asarray(h0, dtype=np.int8).view(np.uint8)
    sc = np.ones(1, np.float32)
    Bm = np.zeros((1, N), np.float32)
    Bm[0, 1:] = fracs
    one = np.ones((1, 1), np.float32)
    for t in range(1, T + 1):
        oracle.state_update(st, sc, fmt, 16, np.ones((1, 1, 1), np.float32), one, np.zeros(1, np.float32), Bm,
                            np.zeros((1, N), np.float32), None, rule, t, weyl_block=16, sr_seed=0)
        assert sc[0] == 1.0
    return st.view(np.int8).reshape(N).astype(np.int64)


@pytest.mark.parametrize("rule", [RTN, SR, WEYL])
@pytest.mark.parametrize("sign", [+1, -1])
def test_proposition_1_identity_on_an_int8_block(rule, sign):
    # Proposition 1 in its native setting (a fixed step): e_T = -s (#{u_t < 1 - f} - T (1 - f))
    T = 100
    fracs = sign * np.array([1, 3, 8, 13, 16, 21, 27, 31, 33, 40, 47, 50, 55, 60, 63]) / 64.0
    h0 = np.full(15, -50 if sign > 0 else 50)
    got = int_recurrence(INT8, fracs.astype(np.float32), h0, T, rule)
    assert got[0] == 127
    m = np.floor(fracs)
    f = fracs - m
    for n in range(15):
        U = [oracle.threshold(rule, flat=n + 1, t=t, weyl_block=16, sr_seed=0) for t in range(1, T + 1)]
        if rule == RTN:
            ups = T if f[n] > 0.5 else 0
        else:
            ups = sum(Fraction(u, 1 << 24) >= 1 - Fraction(float(f[n])) for u in U)
        assert got[n + 1] == h0[n] + T * m[n] + ups
    err = got[1:] - (h0 + T * fracs)
    if rule == RTN:
        assert np.allclose(np.abs(err), T * np.minimum(f, 1 - f))
    elif rule == WEYL:
        assert np.max(np.abs(err)) <= 3.0


@pytest.mark.parametrize("rule", [SR, WEYL])
def test_lemma_2_noise_on_the_uniform_grid(rule):
    rng = np.random.default_rng(4)
    n = 200000
    v = rng.uniform(-100, 100, n).astype(np.float32)
    U = np.array([oracle.threshold(rule, flat=int(i), t=3, weyl_block=16) for i in range(n)], dtype=np.uint32)
    res = oracle.round_values(v, U, INT8, rule).astype(np.float64) - v.astype(np.float64)
    assert abs(np.mean(res**2) - 1 / 6) < 0.004 and abs(np.mean(res)) < 0.004
    res = oracle.round_values(v, 0, INT8, RTN).astype(np.float64) - v.astype(np.float64)
    assert abs(np.mean(res**2) - 1 / 12) < 0.002

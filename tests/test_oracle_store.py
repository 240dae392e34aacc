"""Pins of the oracle's stand-alone store functions and of its sanity metrics.

quantize_store / replay_step: the dither index of entry (row, col) is the flat index of the [-1, row_len] view
that starts `row_index_base` rows into the layer's state, flat = (row_index_base + row) * row_len + col, and block r,
position c of Appendix B "Dithers" are flat / block and flat % block.  Each stored code is rebuilt here element by
element from the separately pinned pieces (threshold, Eq. 2 on the grid, encode), so a dropped or unscaled base fails.

state_error_per_head / readout_kl: the metric of Appendix B "Open-loop replay" and the KL of Section 4
"What we measure", on cases small enough to write the answer out by hand.
"""
from fractions import Fraction
import math

import numpy as np
import pytest

import oracle
from oracle import FP16, BF16, E4M3, FP32, INT8, INT4, RTN, SR, WEYL, SR_HASH

f32 = np.float32
TINY = np.finfo(np.float32).tiny
TOP = {E4M3: 448.0, INT8: 127.0, INT4: 7.0}

# row bases: none, a few rows, and one that carries the flat index past 2^32
BASES = [0, 5, (1 << 32) // 32 + 7]


def _expected_codes(hp, fmt, rule, step_t, base, *, scale_block, weyl_block, layer, weyl_seed, sr_seed):
    """Codes and scales of the FP32 rows `hp` [n_rows, row_len], one entry at a time."""
    n_rows, row_len = hp.shape
    codes = np.zeros(hp.shape, dtype=oracle.CODE_DTYPE[fmt])
    scaled = oracle.has_block_scale(fmt)
    scales = np.zeros((n_rows, row_len // scale_block), f32) if scaled else None
    for row in range(n_rows):
        for col in range(row_len):
            v = hp[row, col]
            if scaled:
                k0 = (col // scale_block) * scale_block
                amax = np.max(np.abs(hp[row, k0:k0 + scale_block]))
                s = max(f32(amax / f32(TOP[fmt])), TINY)
                scales[row, col // scale_block] = s
                v = f32(v * f32(f32(1.0) / s))
            flat = (base + row) * row_len + col
            U = oracle.threshold(rule, flat, step_t, layer=layer, weyl_seed=weyl_seed, weyl_block=weyl_block, sr_seed=sr_seed)
            codes[row, col] = oracle.encode(oracle.round_values(v, U, fmt, rule), fmt)[0]
    return codes, scales


@pytest.mark.parametrize("fmt", [FP16, BF16, E4M3, INT8, INT4])
@pytest.mark.parametrize("rule", [SR, WEYL, SR_HASH])
@pytest.mark.parametrize("base", BASES)
def test_quantize_store_dither_index_follows_row_index_base(fmt, rule, base):
    rng = np.random.default_rng(1000 * fmt + 10 * rule + (base % 7))
    n_rows, row_len = 6, 32
    sb = 16 if oracle.has_block_scale(fmt) else 0
    src = (rng.standard_normal((n_rows, row_len)) * rng.uniform(0.01, 3.0, (n_rows, 1))).astype(f32)
    kw = dict(scale_block=sb, weyl_block=16, layer=3, weyl_seed=2, sr_seed=0x1234567890)
    got_c, got_s = oracle.quantize_store(src, fmt, rule, 7, row_index_base=base, **kw)
    want_c, want_s = _expected_codes(src, fmt, rule, 7, base, **kw)
    assert np.array_equal(got_c, want_c)
    if want_s is not None:
        assert np.array_equal(got_s, want_s)
    # the base matters: the same rows quantised with another base draw other thresholds
    other_c, _ = oracle.quantize_store(src, fmt, rule, 7, row_index_base=base + 1, **kw)
    assert not np.array_equal(other_c, got_c)
    # ... and it is the ROW count that is added: rows 2.. of a store based at `base` are rows 0.. of one based at base + 2
    tail_c, _ = oracle.quantize_store(src[2:], fmt, rule, 7, row_index_base=base + 2, **kw)
    assert np.array_equal(tail_c, got_c[2:])


def test_quantize_store_weyl_block_equal_to_the_row():
    # block = row_len: r is the global row, c the column (the hybrid-shaped configurations)
    rng = np.random.default_rng(77)
    src = rng.standard_normal((4, 64)).astype(f32)
    got, _ = oracle.quantize_store(src, BF16, WEYL, 9, weyl_block=64, layer=1, row_index_base=11)
    for row in range(4):
        for col in range(64):
            U = oracle.weyl_u24(11 + row, col, 1, 0, 9)
            assert got[row, col] == oracle.encode(oracle.round_values(src[row, col], U, BF16, WEYL), BF16)[0]


def _fma32(a, h, w):
    """One fused multiply-add in binary32: exact product and sum, a single rounding."""
    return f32(float(Fraction(float(a)) * Fraction(float(h)) + Fraction(float(w))))


@pytest.mark.parametrize("fmt", [FP16, BF16, E4M3, INT8])
@pytest.mark.parametrize("rule", [SR, WEYL, SR_HASH])
@pytest.mark.parametrize("base", BASES)
def test_replay_step_dither_index_follows_row_index_base(fmt, rule, base):
    rng = np.random.default_rng(2000 * fmt + 10 * rule + (base % 7))
    n_rows, row_len, rpd = 4, 32, 2
    sb = 16 if oracle.has_block_scale(fmt) else 0
    kw = dict(scale_block=sb, weyl_block=16, layer=1, weyl_seed=4, sr_seed=99)
    h0 = rng.standard_normal((n_rows, row_len)).astype(f32)
    codes, scales = oracle.quantize_store(h0, fmt, RTN, 1, scale_block=sb)
    w = (0.3 * rng.standard_normal((n_rows, row_len))).astype(f32)
    a = rng.uniform(0.5, 1.0, n_rows // rpd).astype(f32)
    h_in = oracle.decode(codes, fmt)
    if scales is not None:
        h_in = (h_in.reshape(n_rows, -1, sb) * scales[:, :, None]).astype(f32).reshape(n_rows, row_len)
    hp = np.array([[_fma32(a[r // rpd], h_in[r, c], w[r, c]) for c in range(row_len)] for r in range(n_rows)], dtype=f32)
    want_c, want_s = _expected_codes(hp, fmt, rule, 12, base, **kw)
    got_c = codes.copy()
    got_s = None if scales is None else scales.copy()
    oracle.replay_step(w, a, rpd, got_c, got_s, fmt, rule, 12, row_index_base=base, **kw)
    assert np.array_equal(got_c, want_c)
    if want_s is not None:
        assert np.array_equal(got_s, want_s)
    other = codes.copy()
    oracle.replay_step(w, a, rpd, other, None if scales is None else scales.copy(), fmt, rule, 12, row_index_base=base + 1, **kw)
    assert not np.array_equal(other, got_c)


# ---- sanity metrics, by hand -----------------------------------------------------------------------
def test_state_error_per_head_on_a_case_written_out_by_hand():
    # B = 2, H = 2, P = 1, N = 16, FP16 codes (every value below is an FP16 number).  Head 0: the store equals the
    # twin except for two entries off by 1/4 and 1/2; head 1: every entry of the store is the twin's plus 1/8.
    B, H, P, N = 2, 2, 1, 16
    twin = np.zeros((B, H, P, N), f32)
    twin[0, 0, 0, :] = 1.0                       # sum of squares 16
    twin[1, 0, 0, :] = 2.0                       # 64
    twin[0, 1, 0, :] = 0.5                       # 4
    twin[1, 1, 0, :] = -1.0                      # 16
    stored = twin.copy()
    stored[0, 0, 0, 3] += 0.25                   # 1/16
    stored[1, 0, 0, 9] -= 0.5                    # 1/4
    stored[:, 1] += 0.125                        # 32 entries * 1/64 = 1/2
    codes = oracle.encode(stored, FP16)
    err2, ref2 = oracle.state_error_per_head(codes, None, twin, FP16)
    assert err2.tolist() == [1 / 16 + 1 / 4, 0.5]
    assert ref2.tolist() == [80.0, 20.0]
    # a scaled store: INT8 codes k with one scale per row, h_hat = k * s
    k = np.zeros((B, H, P, N), np.int8)
    k[0, 0, 0, 0], k[1, 1, 0, 5] = 127, -64
    scales = np.array([0.5, 1.0, 1.0, 0.25], f32)              # rows (b, h) = (0,0), (0,1), (1,0), (1,1)
    tw = np.zeros((B, H, P, N), f32)
    tw[0, 0, 0, 0], tw[1, 1, 0, 5] = 63.0, -15.0               # h_hat = 63.5 and -16
    err2, ref2 = oracle.state_error_per_head(k.view(np.uint8), scales, tw, INT8, 16)
    assert err2.tolist() == [0.25, 1.0]
    assert ref2.tolist() == [63.0**2, 225.0]


def test_readout_kl_on_a_case_written_out_by_hand():
    ln2 = math.log(2.0)
    # sequence 0: p = softmax(0, ln 2) = (1/3, 2/3), q = softmax(0, 0) = (1/2, 1/2)
    # sequence 1: p = (1/2, 1/4, 1/4), q = (1/4, 1/4, 1/2), given as log-weights with an arbitrary common shift
    y_ref = np.array([[0.0, ln2, -1e30], [3.0 + ln2, 3.0, 3.0]])
    y_q = np.array([[7.0, 7.0, -1e30], [-1.0, -1.0, -1.0 + ln2]])
    got = oracle.readout_kl(y_ref, y_q)
    want0 = (1 / 3) * math.log((1 / 3) / (1 / 2)) + (2 / 3) * math.log((2 / 3) / (1 / 2))
    want1 = 0.5 * math.log(2.0) + 0.25 * math.log(1.0) + 0.25 * math.log(0.5)
    assert got == pytest.approx([want0, want1], rel=1e-12)
    assert np.all(oracle.readout_kl(y_ref, y_ref) == 0.0)
    # not symmetric: KL(q || p) is another number
    assert oracle.readout_kl(y_q, y_ref)[0] == pytest.approx(0.5 * math.log(0.5 / (1 / 3)) + 0.5 * math.log(0.5 / (2 / 3)), rel=1e-12)
    # shape: any trailing dimensions are flattened per sequence
    assert oracle.readout_kl(y_ref.reshape(2, 3, 1), y_q.reshape(2, 3, 1)) == pytest.approx([want0, want1], rel=1e-12)


# ---- one scale per (sequence, head): scale_block = P * N ---------------------------------------------------------
@pytest.mark.parametrize("fmt", [E4M3, INT8])
@pytest.mark.parametrize("rule", [RTN, WEYL, SR])
def test_head_scale_step_against_an_element_by_element_restatement(fmt, rule):
    """Section 2 "Low-precision storage" defines s = max|h| / top over a block; here the block is the whole head.  The
    step is rebuilt from the pinned pieces: FP32 update, one scale from the head's maximum, v = h' * (1/s), threshold of
    the flat index, Eq. 2, encode."""
    rng = np.random.default_rng(300 + 10 * fmt + rule)
    Bsz, H, P, N = 2, 3, 4, 32
    sb = P * N
    A = -np.exp(rng.uniform(-3, 1, H)).astype(f32)
    state = rng.integers(-7, 8, (Bsz, H, P, N)).astype(np.int8).view(np.uint8) if fmt == INT8 else \
        oracle.encode((rng.standard_normal((Bsz, H, P, N)) * 20).astype(f32), E4M3)
    scales = rng.uniform(0.01, 0.2, Bsz * H).astype(f32)
    x = rng.standard_normal((Bsz, H, P)).astype(f32)
    dt = np.log1p(np.exp(rng.normal(-2, 0.5, (Bsz, H)))).astype(f32)
    Bm = rng.standard_normal((Bsz, N)).astype(f32)
    Cm = rng.standard_normal((Bsz, N)).astype(f32)
    base, t = 5, 9
    want_codes = np.zeros_like(state)
    want_scales = np.zeros_like(scales)
    want_y = np.zeros((Bsz, H, P))
    for b in range(Bsz):
        for h in range(H):
            a = oracle.exp_spec(f32(dt[b, h] * A[h]))[0]
            h_in = (oracle.decode(state[b, h], fmt) * scales[b * H + h]).astype(f32)
            hp = np.zeros((P, N), f32)
            for p in range(P):
                dtx = f32(dt[b, h] * x[b, h, p])
                for n in range(N):
                    hp[p, n] = _fma32(a, h_in[p, n], f32(dtx * Bm[b, n]))
                want_y[b, h, p] = float(np.dot(Cm[b].astype(np.float64), hp[p].astype(np.float64)))
            s = max(f32(np.max(np.abs(hp)) / f32(TOP[fmt])), TINY)
            want_scales[b * H + h] = s
            rinv = f32(f32(1.0) / s)
            for p in range(P):
                for n in range(N):
                    flat = ((((base + b) * H + h) * P + p) * N + n)
                    U = oracle.threshold(rule, flat, t, layer=1, weyl_seed=0, weyl_block=16, sr_seed=77)
                    want_codes[b, h, p, n] = oracle.encode(oracle.round_values(f32(hp[p, n] * rinv), U, fmt, rule), fmt)[0]
    y = oracle.state_update(state, scales, fmt, sb, x, dt, A, Bm, Cm, None, rule, t, layer=1, weyl_block=16, sr_seed=77,
                            batch_index_base=base)
    assert np.array_equal(state, want_codes)
    assert np.array_equal(scales, want_scales)
    assert np.allclose(y, want_y, rtol=0, atol=1e-6 * np.max(np.abs(want_y)))
    top_code = int(TOP[fmt]) if fmt == INT8 else 0x7E
    mags = state.view(np.int8).astype(np.int32) if fmt == INT8 else (state & 0x7F).astype(np.int32)
    assert np.all(np.abs(mags).reshape(Bsz * H, -1).max(axis=1) >= top_code - 1)       # the head's maximum lands on the top


def test_head_scale_absorbs_a_shared_decay():
    # one decay per head and no write: the single FP32 scale carries the decay and, under RTN, every code of the head stays
    rng = np.random.default_rng(6)
    Bsz, H, P, N = 1, 2, 4, 128
    src = rng.standard_normal((Bsz * H, P * N)).astype(f32)
    state = np.zeros((Bsz, H, P, N), np.uint8)
    scales = np.zeros(Bsz * H, f32)
    for i in range(Bsz * H):                     # quantise each head as one block of P * N entries
        s = max(f32(np.max(np.abs(src[i])) / f32(448.0)), TINY)
        scales[i] = s
        state.reshape(Bsz * H, -1)[i] = oracle.round_encode((src[i] * f32(f32(1.0) / s)).astype(f32), None, E4M3, RTN)
    before, s_before = state.copy(), scales.copy()
    A = np.array([-0.5, -0.01], f32)
    zero = np.zeros((Bsz, N), f32)
    for t in range(1, 20):
        oracle.state_update(state, scales, E4M3, P * N, np.zeros((Bsz, H, P), f32), np.full((Bsz, H), 0.1, f32), A, zero, zero,
                            None, RTN, t, weyl_block=128)
    assert np.array_equal(state, before)
    assert np.allclose(scales / s_before, np.exp(0.1 * A.astype(np.float64)) ** 19, rtol=1e-5)


def test_block_scale_is_the_ieee_quotient_floored_at_the_smallest_normal():
    """s = max|h'| / top in FP32 (Appendix B "Formats"): against the quotient taken in double and rounded once (a double
    quotient of two binary32 numbers rounds to the binary32 quotient: 53 >= 2 * 24 + 2), for random maxima, powers of
    two, subnormals and zero, each format's top."""
    rng = np.random.default_rng(3)
    amax = np.concatenate([np.abs(rng.standard_normal(4000)).astype(np.float32) * np.float32(10.0) ** rng.integers(-38, 38, 4000).astype(np.float32),
                           np.float32(2.0) ** np.arange(-149, 128, dtype=np.float32), np.zeros(1, np.float32),
                           rng.integers(1, 1 << 23, 500).astype(np.uint32).view(np.float32)])
    amax = amax[np.isfinite(amax)]
    tiny = np.float32(np.finfo(np.float32).tiny)
    for fmt, top in ((oracle.E4M3, 448.0), (oracle.INT8, 127.0), (oracle.INT7, 63.0), (oracle.INT6, 31.0), (oracle.INT4, 7.0)):
        want = np.maximum((amax.astype(np.float64) / top).astype(np.float32), tiny)
        assert np.array_equal(oracle.block_scale(amax, fmt), want)

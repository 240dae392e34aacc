"""Pins of the oracle's threshold generators against what the paper and the mathematics fix."""
import math
import os

import numpy as np
import pytest

import oracle

NO_OFFSET = 0xFFFFFFFF   # r + 1 == c + 1 == 0 (mod 2^32): the accumulator reduces to t * Phi
PHI = 2654435769
ALPHA = (math.sqrt(5.0) - 1.0) / 2.0


def star_discrepancy(u):
    """D*_T of a point set in [0,1): sup_x |A_T(x)/T - x| from the sorted points (Appendix A)."""
    u = np.sort(np.asarray(u, dtype=np.float64))
    T = len(u)
    i = np.arange(1, T + 1)
    return max(np.max(i / T - u), np.max(u - (i - 1) / T))


def test_weyl_sequence_starts_618_236_854():
    # Introduction: the Weyl thresholds are 0.618, 0.236, 0.854, ... (first write is t = 1)
    got = [oracle.weyl_u24(NO_OFFSET, NO_OFFSET, 0, 0, t) / 2.0**24 for t in (1, 2, 3)]
    assert [round(g, 3) for g in got] == [0.618, 0.236, 0.854]
    assert [oracle.weyl_u24(NO_OFFSET, NO_OFFSET, 0, 0, t) for t in (1, 2, 3)] == [10368889, 3960563, 14329453]
    for t, g in zip((1, 2, 3), got):
        assert abs(g - (t * ALPHA) % 1.0) < 2.0**-23


def test_weyl_integer_form_tracks_float_form():
    # Appendix B "Dithers": u = frac(o_{r,c} + t*alpha) with the decimal generators; the 32-bit
    # accumulator holds each generator scaled by 2^32 and rounded, so each term is off by at most half a unit of 2^-32.
    rng = np.random.default_rng(0)
    for _ in range(2000):
        r, c = int(rng.integers(0, 1 << 20)), int(rng.integers(0, 128))
        layer, seed, t = int(rng.integers(0, 64)), int(rng.integers(0, 4)), int(rng.integers(1, 1 << 16))
        u_int = oracle.weyl_u24(r, c, layer, seed, t) / 2.0**24
        o = math.fmod(0.7548776662 * (r + 1), 1.0) + math.fmod(0.5698402910 * (c + 1), 1.0) \
            + math.fmod(0.1234567 * layer, 1.0) + math.fmod(0.3141592 * seed, 1.0)
        u_flt = (o + math.fmod(t * ALPHA, 1.0)) % 1.0          # phase reduced modulo 1 in float64 first
        d = abs(u_int - u_flt)
        d = min(d, 1.0 - d)
        assert d <= 2.0**-24 + 2.0**-33 * ((r + 1) + (c + 1) + layer + seed + t) + 1e-9


def test_accumulator_is_linear_mod_2_32():
    # definition check on independent arithmetic (Python big integers)
    rng = np.random.default_rng(1)
    A, B, L, S = 3242174889, 2447445414, 530242489, 1349303490
    assert A == round(0.7548776662 * 2**32) and B == round(0.5698402910 * 2**32)
    assert L == round(0.1234567 * 2**32) and S == round(0.3141592 * 2**32)
    assert PHI == round(ALPHA * 2**32)
    for _ in range(1000):
        r, c, l, s, t = (int(v) for v in rng.integers(0, 1 << 32, 5))
        want = (A * (r + 1) + B * (c + 1) + L * l + S * s + t * PHI) % 2**32
        assert oracle.weyl_acc(r, c, l, s, t) == want


def test_knuth_offsets_alias_but_r2_offsets_do_not():
    # Observation 1: with the row multiplier equal (up to 8 * 2^-32) to Phi, entry i+1 at step t gets
    # the threshold of entry i at step t+1 except where a carry crosses the dropped 8 bits.
    H = 2654435761
    assert PHI - H == 8
    same = 0
    total = 0
    for i in range(64):
        for t in range(1, 257):
            a = (((i + 2) * H + t * PHI) % 2**32) >> 8
            b = (((i + 1) * H + (t + 1) * PHI) % 2**32) >> 8
            same += (a == b)
            total += 1
    assert same / total > 0.95
    # the oracle's generators: no coincidence between neighbours at any small lag
    worst = 1.0
    for dr in range(-2, 3):
        for dc in range(-2, 3):
            if dr == 0 and dc == 0:
                continue
            for lag in range(-16, 17):
                a = oracle.weyl_acc(10 + dr, 10 + dc, 0, 0, 100 + lag)
                b = oracle.weyl_acc(10, 10, 0, 0, 100)
                d = ((a - b) % 2**32) / 2.0**32
                worst = min(worst, d, 1.0 - d)
    # Appendix B "Offset near-aliasing": separation d = 0.0015 for these generators
    assert 0.0012 < worst < 0.0018


def test_integer_phase_keeps_all_streams_distinct():
    # Observation 2: a float32 phase leaves at most 8192 / 2048 / 512 distinct streams at
    # t = 2047 / 8191 / 32767; the integer accumulator keeps every entry's stream distinct.
    n = 32768
    r = np.arange(n, dtype=np.uint64) // 16
    c = np.arange(n, dtype=np.uint64) % 16
    off = (3242174889 * (r + 1) + 2447445414 * (c + 1)) % 2**32
    for t, limit in ((2047, 8192), (8191, 2048), (32767, 512)):
        acc = (off + t * PHI) % 2**32
        spot = [oracle.weyl_acc(int(r[i]), int(c[i]), 0, 0, t) for i in (0, 1, 17, n - 1)]
        assert spot == [int(acc[i]) for i in (0, 1, 17, n - 1)]
        assert len(np.unique(acc)) == n
        o32 = (off.astype(np.float64) / 2.0**32).astype(np.float32)
        phase32 = o32 + np.float32(t) * np.float32(ALPHA)          # the defective float32 phase
        frac = phase32 - np.floor(phase32)
        assert len(np.unique(frac)) <= limit


def test_local_discrepancy_matches_table_8():
    # Table 8: LD_256 = 0.0078 (Weyl, alpha = phi - 1) and 0.0539 (SR); Appendix B "Dithers" defines
    # it as the mean star discrepancy of 256 consecutive thresholds over random starts and offsets.
    rng = np.random.default_rng(2)
    vals = []
    for _ in range(64):
        r, c = int(rng.integers(0, 1 << 16)), int(rng.integers(0, 16))
        t0 = int(rng.integers(1, 1 << 20))
        u = [oracle.weyl_u24(r, c, 0, 0, t0 + k) / 2.0**24 for k in range(256)]
        vals.append(star_discrepancy(u))
    assert abs(np.mean(vals) - 0.0078) < 0.0008
    vals = []
    for j in range(200):
        u = [oracle.threshold(oracle.SR, flat=1000 + j, t=t, sr_seed=0) / 2.0**24 for t in range(1, 257)]
        vals.append(star_discrepancy(u))
    assert abs(np.mean(vals) - 0.0539) < 0.004


def test_weyl_discrepancy_grows_like_log_T():
    # Corollary 1(c): T * D*_T of the golden-ratio sequence stays O(log T)
    for T, bound in ((64, 2.5), (1024, 3.0), (4096, 3.5)):
        u = [oracle.weyl_u24(NO_OFFSET, NO_OFFSET, 0, 0, t) / 2.0**24 for t in range(1, T + 1)]
        assert T * star_discrepancy(u) < bound


def test_philox_known_answers(golden_dir):
    n = 0
    for line in open(os.path.join(golden_dir, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        ctr, key, out = ([int(w, 16) for w in part.split()] for part in line.split("|"))
        assert list(oracle.philox4x32_10(ctr, key)) == out
        n += 1
    assert n == 3


def test_sr_counter_layout():
    # four consecutive entries share one Philox call: counter = (flat/4 lo, flat/4 hi, t, layer), word flat%4
    for flat in (0, 5, 2**34 + 7):
        for t, layer, seed in ((1, 0, 0), (77, 3, 0x123456789A)):
            g = flat // 4
            out = oracle.philox4x32_10([g & 0xFFFFFFFF, g >> 32, t, layer], [seed & 0xFFFFFFFF, seed >> 32])
            assert oracle.threshold(oracle.SR, flat, t, layer=layer, sr_seed=seed) == int(out[flat % 4]) >> 8


def test_sr_thresholds_look_uniform():
    # the paper's acceptance numbers for its SR source: mean 0.4997, variance 0.0834, lag-1 correlation -5e-5
    n = 40000
    u = np.array([oracle.threshold(oracle.SR, flat=12345, t=t, sr_seed=0) for t in range(1, n + 1)]) / 2.0**24
    assert abs(u.mean() - 0.5) < 3 * math.sqrt(1 / 12 / n)
    assert abs(u.var() - 1 / 12) < 0.002
    lag1 = np.corrcoef(u[:-1], u[1:])[0, 1]
    assert abs(lag1) < 3 / math.sqrt(n)
    across = np.array([oracle.threshold(oracle.SR, flat=f, t=9, sr_seed=1) for f in range(n)]) / 2.0**24
    assert abs(across.mean() - 0.5) < 3 * math.sqrt(1 / 12 / n)
    assert abs(np.corrcoef(across[:-1], across[1:])[0, 1]) < 3 / math.sqrt(n)


# ---- integer-hash SR ---------------------------------------------------------------------------
def _unfmix32(h):
    """Inverse of the MurmurHash3 finaliser, built from the modular inverses of its two multipliers and the
    inverses of its xor-shifts (different operations from the forward direction)."""
    m = 0xFFFFFFFF
    h ^= h >> 16
    h = (h * pow(0xC2B2AE35, -1, 2**32)) & m
    h ^= (h >> 13) ^ (h >> 26)
    h = (h * pow(0x85EBCA6B, -1, 2**32)) & m
    h ^= h >> 16
    return h


def test_fmix32_is_the_murmur3_finaliser():
    rng = np.random.default_rng(11)
    assert oracle.fmix32(0) == 0
    xs = [int(v) for v in rng.integers(0, 1 << 32, 3000)] + [1, 2, 0xFFFFFFFF, 0x80000000]
    for x in xs:
        assert _unfmix32(oracle.fmix32(x)) == x                       # a permutation, inverted by independent arithmetic
    # avalanche: flipping one input bit flips about half of the output bits
    flips = []
    for x in xs[:300]:
        for b in (0, 7, 16, 31):
            flips.append(bin(oracle.fmix32(x) ^ oracle.fmix32(x ^ (1 << b))).count("1"))
    assert 15.0 < np.mean(flips) < 17.0


def test_hash_sr_definition_and_moments():
    # definition: fmix32(i_lo*P1 + t*P2 + layer*P3 + seed_lo*P4 + (i_hi ^ seed_hi)*P5) >> 8 with the two multipliers
    # the paper prints (0x9E3779B1 for the entry, 0x85EBCA77 for the step)
    P1, P2, P3, P4, P5 = 0x9E3779B1, 0x85EBCA77, 0xC2B2AE3D, 0x27D4EB2F, 0x165667B1
    for flat, t, layer, seed in ((0, 1, 0, 0), (12345, 99, 3, 7), (2**35 + 17, 2**31 + 5, 11, 2**40 + 3)):
        key = ((flat & 0xFFFFFFFF) * P1 + t * P2 + layer * P3 + (seed & 0xFFFFFFFF) * P4 + ((flat >> 32) ^ (seed >> 32)) * P5) % 2**32
        assert oracle.threshold(oracle.SR_HASH, flat, t, layer=layer, sr_seed=seed) == oracle.fmix32(key) >> 8
    # the paper's unit test of its hash: mean 0.4997, variance 0.0834, lag-1 correlation -5e-5
    n = 40000
    u = np.array([oracle.threshold(oracle.SR_HASH, flat=777, t=t) for t in range(1, n + 1)]) / 2.0**24
    assert abs(u.mean() - 0.5) < 3 * math.sqrt(1 / 12 / n)
    assert abs(u.var() - 1 / 12) < 0.002
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 3 / math.sqrt(n)
    across = np.array([oracle.threshold(oracle.SR_HASH, flat=f, t=5) for f in range(n)]) / 2.0**24
    assert abs(across.mean() - 0.5) < 3 * math.sqrt(1 / 12 / n)
    assert abs(np.corrcoef(across[:-1], across[1:])[0, 1]) < 3 / math.sqrt(n)
    # local discrepancy of a random sequence (Table 8, row SR: 0.0539)
    vals = [star_discrepancy([oracle.threshold(oracle.SR_HASH, flat=2000 + j, t=t) / 2.0**24 for t in range(1, 257)])
            for j in range(200)]
    assert abs(np.mean(vals) - 0.0539) < 0.004


def test_discrepancy_utility_reproduces_table_8_for_other_increments():
    """The star-discrepancy utility used by the pins above, checked on sequences the oracle does not implement:
    LD_256 of Weyl dithers with other increments (Table 8), float64 phase reduced modulo 1."""
    phi = (1 + math.sqrt(5)) / 2
    rows = {"sqrt2-1": (math.sqrt(2) - 1, 0.0069), "1/(2+phi)": (1 / (2 + phi), 0.0075), "e-2": (math.e - 2, 0.0097),
            "1/4+2^-12": (0.25 + 2.0**-12, 0.1379), "1/3+2^-12": (1 / 3 + 2.0**-12, 0.2063), "1/2+2^-12": (0.5 + 2.0**-12, 0.3347)}
    rng = np.random.default_rng(12)
    for name, (alpha, want) in rows.items():
        vals = []
        for _ in range(400):      # more starts than the paper's 64: the near-rational rows vary strongly with the offset
            o, t0 = rng.random(), int(rng.integers(1, 1 << 20))
            u = (o + (np.arange(t0, t0 + 256) * alpha) % 1.0) % 1.0
            vals.append(star_discrepancy(u))
        assert abs(np.mean(vals) - want) < max(0.0008, 0.06 * want), name


def test_near_rational_increment_is_as_bad_as_rtn():
    # Corollary 1(d): alpha = 1/2 + eps leaves two empty arcs of length 3/8 for T <= 1/(8 eps): D*_T >= 3/16
    eps = 2.0**-12
    T = int(1 / (8 * eps))
    for o in (0.0, 0.3, 0.77):
        u = (o + np.arange(1, T + 1) * (0.5 + eps)) % 1.0
        assert star_discrepancy(u) >= 3 / 16 - 1e-9
    # while the golden-ratio sequence of the same length is two orders of magnitude more even
    u = np.array([oracle.weyl_u24(NO_OFFSET, NO_OFFSET, 0, 0, t) for t in range(1, T + 1)]) / 2.0**24
    assert star_discrepancy(u) < 0.01

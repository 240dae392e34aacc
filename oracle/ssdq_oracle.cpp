// ssdq_oracle.cpp -- TEST INFRASTRUCTURE ONLY.
//
// Plain, slow, single-pass-per-entry CPU statement of the quantized selective-state-update decode
// step and its three rounding rules, written from the paper ("Low-Discrepancy Dither for Quantized
// Recurrent State Caches").  It exists so that the CUDA library can be checked against something
// that a reader can compare with the paper by eye.  It shares no code, header, table or constant
// generator with the CUDA path and must never be imported, linked or called by the product: only
// the tests, the smoke check and the CPU-baseline leg of the benchmark may use it.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fopenmp -shared -fPIC   (no -ffast-math: every
// float operation below is meant to be one IEEE-754 binary32 operation, fused only where fmaf is
// written out).
//
// What follows the paper and where:
//   * recurrence h_t = a_t h_{t-1} + w_t                       -- Eq. 1
//   * a = exp(A * dt), w = dt * x (outer) B                      -- Appendix B "Runners", "Open-loop replay"
//   * FP32 update, rounding only on write-back                 -- Section 2 "Low-precision storage"
//   * Q_u(x) = s * floor(x / s + u) on the local grid           -- Eq. 2 and the sentence after it
//   * RTN / SR / Weyl thresholds                                -- Section 2 "Rounding with a threshold"
//   * 32-bit Weyl accumulator, top 24 bits, R2 offsets          -- Appendix B "Dithers"
//   * FP16 / BF16 / FP8-E4M3 + FP32 block scale max|h| / 448    -- Appendix B "Formats"
//   * INT8/7/6/4 symmetric block-absmax, FP32 scale, clamp     -- Appendix B "Formats" (INTb)
//
// Pins (tests/test_oracle_*.py): Weyl 0.618, 0.236, 0.854; Philox known answers; RTN equal to
// library casts; dithered rounding equal to exact rational arithmetic; Proposition 1 identity,
// Lemma 1, Lemma 2, Observations 1 and 2; LD_256 of Table 8; closed form of Eq. 1 without rounding.
// Parity unpinned: the paper's own SR random stream and its own numbering of blocks r cannot be
// recovered from the text; the readings taken here are listed in the design notes of the repo.

#include <algorithm>
#include <cfenv>
#include <cfloat>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum Format { FMT_FP16 = 0, FMT_BF16 = 1, FMT_E4M3 = 2, FMT_FP32 = 3 /* no rounding: the fp32-state twin */,
              FMT_INT8 = 4, FMT_INT7 = 5, FMT_INT6 = 6, FMT_INT4 = 7 /* symmetric block-absmax integers in an int8 container */ };
enum Rule { RULE_RTN = 0, RULE_SR = 1, RULE_WEYL = 2, RULE_SR_HASH = 3 };

struct FormatSpec {
    int mant_bits;   // explicit mantissa bits m
    int e_min;       // exponent of the smallest normal number
    int bias;        // exponent bias of the stored field
    int exp_bits;
    double max_finite;
};

// Appendix B "Formats": E4M3 has 3 mantissa bits, minimum exponent -6, subnormals, saturation at 448.
// FP16 and BF16 are the IEEE binary16 layout and the top half of binary32.
FormatSpec spec_of(int fmt) {
    switch (fmt) {
        case FMT_FP16: return {10, -14, 15, 5, 65504.0};
        case FMT_BF16: return {7, -126, 127, 8, std::ldexp(255.0, 120)};  // (2 - 2^-7) * 2^127
        case FMT_E4M3: return {3, -6, 7, 4, 448.0};
        default:       return {23, -126, 127, 8, (double)FLT_MAX};
    }
}

// Appendix B "Formats", INTb: symmetric, q_max = 2^(b-1) - 1, block scale s = max|h| / q_max kept in FP32,
// values clamped to [-q_max, q_max].  The grid is uniform (step 1 in units of s), so Eq. 2 is floor(v + u).
bool is_int_format(int fmt) { return fmt >= FMT_INT8 && fmt <= FMT_INT4; }
int int_qmax(int fmt) {
    switch (fmt) { case FMT_INT8: return 127; case FMT_INT7: return 63; case FMT_INT6: return 31; default: return 7; }
}
bool has_block_scale(int fmt) { return fmt == FMT_E4M3 || is_int_format(fmt); }

// ------------------------------------------------------------------------------------------
// Thresholds.  U is a 24-bit integer, the leading 24 bits of the 32-bit accumulator, and u = U / 2^24
// (Appendix B "Dithers").
// ------------------------------------------------------------------------------------------

// Appendix B "Dithers", hardware form.  The four multipliers are the decimal constants printed
// there times 2^32, rounded to the nearest integer; Phi is printed as an integer.
const uint32_t WEYL_A = 3242174889u;    // 0.7548776662 * 2^32
const uint32_t WEYL_B = 2447445414u;    // 0.5698402910 * 2^32
const uint32_t WEYL_L = 530242489u;     // 0.1234567    * 2^32
const uint32_t WEYL_S = 1349303490u;    // 0.3141592    * 2^32
const uint32_t WEYL_PHI = 2654435769u;  // golden-ratio increment in 32-bit fixed point

uint32_t weyl_acc(uint32_t r, uint32_t c, uint32_t layer, uint32_t seed, uint32_t t) {
    // all arithmetic modulo 2^32 (unsigned wrap-around)
    return WEYL_A * (r + 1u) + WEYL_B * (c + 1u) + WEYL_L * layer + WEYL_S * seed + t * WEYL_PHI;
}

// Philox4x32 with 10 rounds, from its published definition (Salmon et al., "Parallel random
// numbers: as easy as 1, 2, 3", 2011): two 32x32->64 multiplies per round, key bumped by the
// two Weyl constants between rounds.
void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Integer-hash SR (Section 6.5 "Cost": SR driven by a cheap integer hash is as accurate as Philox SR; Appendix B
// "Decode regime": the hash fmix32(i * 0x9E3779B1 + t * 0x85EBCA77 + ...), of which 24 bits are kept).  fmix32 is the
// 32-bit finaliser of MurmurHash3.  The paper elides the remaining terms; this build continues the same family
// of odd multipliers for layer and seed and folds in the high half of a 64-bit entry index.
uint32_t fmix32(uint32_t h) {
    h ^= h >> 16;
    h *= 0x85EBCA6Bu;
    h ^= h >> 13;
    h *= 0xC2B2AE35u;
    h ^= h >> 16;
    return h;
}
uint32_t hash_sr_word(uint64_t flat, uint32_t t, uint32_t layer, uint64_t seed) {
    const uint32_t i_lo = (uint32_t)flat, i_hi = (uint32_t)(flat >> 32);
    const uint32_t s_lo = (uint32_t)seed, s_hi = (uint32_t)(seed >> 32);
    return fmix32(i_lo * 0x9E3779B1u + t * 0x85EBCA77u + layer * 0xC2B2AE3Du + s_lo * 0x27D4EB2Fu + (i_hi ^ s_hi) * 0x165667B1u);
}

struct RuleParams {
    int rule;
    uint32_t layer;       // layer index l (Weyl offsets and SR counter)
    uint32_t weyl_seed;   // sigma
    uint32_t weyl_block;  // entries per dither block: r = flat / block, c = flat % block
    uint64_t sr_seed;     // Philox key
};

// Threshold of entry `flat` (flat index in the layer's [B_global, H, P, N] state tensor) at write t.
uint32_t threshold_u24(const RuleParams& rp, uint64_t flat, uint32_t t) {
    if (rp.rule == RULE_WEYL) {
        uint32_t r = (uint32_t)(flat / rp.weyl_block);   // block index, taken modulo 2^32
        uint32_t c = (uint32_t)(flat % rp.weyl_block);   // position inside the block
        return weyl_acc(r, c, rp.layer, rp.weyl_seed, t) >> 8;
    }
    if (rp.rule == RULE_SR) {
        uint64_t g = flat / 4;  // one Philox call serves four consecutive entries
        uint32_t ctr[4] = {(uint32_t)g, (uint32_t)(g >> 32), t, rp.layer};
        uint32_t key[2] = {(uint32_t)rp.sr_seed, (uint32_t)(rp.sr_seed >> 32)};
        uint32_t out[4];
        philox4x32_10(ctr, key, out);
        return out[flat % 4] >> 8;
    }
    if (rp.rule == RULE_SR_HASH) return hash_sr_word(flat, t, rp.layer, rp.sr_seed) >> 8;
    return 0;  // RTN has no threshold
}

// ------------------------------------------------------------------------------------------
// Rounding on the local grid (Eq. 2): Q = 2^q * floor(v / 2^q + u) with 2^q the spacing of the
// target format at |v| (subnormal-aware); RTN is round-to-nearest with ties to even, the rule
// of the native casts which the paper says its simulation reproduces bit for bit.
// All intermediate values are exact in double: v / 2^q has at most 24 significant bits, u is a
// multiple of 2^-24, and their sum needs at most 53 bits whenever it can reach or pass an integer.
// ------------------------------------------------------------------------------------------
float round_on_grid(float v, int fmt, int rule, uint32_t U) {
    if (fmt == FMT_FP32) return v;
    if (is_int_format(fmt)) {
        if (std::isnan(v)) return v;
        const double q = (double)int_qmax(fmt);
        if (std::isinf(v)) return (float)std::copysign(q, (double)v);
        // v has at most 24 significant bits and u is a multiple of 2^-24: the sum is exact in double
        double K = (rule == RULE_RTN) ? std::nearbyint((double)v) : std::floor((double)v + std::ldexp((double)U, -24));
        K = std::min(std::max(K, -q), q);
        return (float)(K == 0.0 ? 0.0 : K);   // an integer zero has no sign
    }
    const FormatSpec fs = spec_of(fmt);
    if (std::isnan(v)) return v;
    if (std::isinf(v)) return std::copysign((float)fs.max_finite, v);
    if (v == 0.0f) return v;  // +0 stays +0, -0 stays -0
    int ex;
    std::frexp((double)v, &ex);  // |v| = f * 2^ex with f in [0.5, 1)  =>  floor(log2 |v|) = ex - 1
    const int e = ex - 1;
    const int q = std::max(e, fs.e_min) - fs.mant_bits;
    const double g = std::ldexp((double)v, -q);  // exact
    double K;
    if (rule == RULE_RTN) {
        K = std::nearbyint(g);  // FE_TONEAREST: ties to even
    } else {
        K = std::floor(g + std::ldexp((double)U, -24));
    }
    double Q = std::ldexp(K, q);  // exact
    if (std::fabs(Q) > fs.max_finite) Q = std::copysign(fs.max_finite, (double)v);
    float out = (float)Q;  // exact: Q is on the target grid, a subset of binary32
    if (out == 0.0f) out = std::copysign(0.0f, v);  // a value that rounds to zero keeps its sign
    return out;
}

// Storage codes, from the bit layout of each format.
uint32_t encode(float q, int fmt) {
    const FormatSpec fs = spec_of(fmt);
    if (fmt == FMT_FP32) { uint32_t b; std::memcpy(&b, &q, 4); return b; }
    if (is_int_format(fmt)) return (uint32_t)(uint8_t)(int8_t)(int)q;   // two's complement byte
    const uint32_t sign = std::signbit(q) ? 1u : 0u;
    const int total_bits = 1 + fs.exp_bits + fs.mant_bits;
    uint32_t field_e = 0, field_m = 0;
    const double a = std::fabs((double)q);
    if (std::isnan(q)) {
        field_e = (1u << fs.exp_bits) - 1u; field_m = (1u << fs.mant_bits) - 1u;
    } else if (a != 0.0) {
        int ex;
        std::frexp(a, &ex);
        const int e = ex - 1;
        if (e >= fs.e_min) {
            field_e = (uint32_t)(e + fs.bias);
            field_m = (uint32_t)std::ldexp(a - std::ldexp(1.0, e), fs.mant_bits - e);
        } else {
            field_e = 0;
            field_m = (uint32_t)std::ldexp(a, fs.mant_bits - fs.e_min);
        }
    }
    return (sign << (total_bits - 1)) | (field_e << fs.mant_bits) | field_m;
}

float decode(uint32_t code, int fmt) {
    if (fmt == FMT_FP32) { float f; std::memcpy(&f, &code, 4); return f; }
    if (is_int_format(fmt)) return (float)(int8_t)(uint8_t)code;
    const FormatSpec fs = spec_of(fmt);
    const int total_bits = 1 + fs.exp_bits + fs.mant_bits;
    const uint32_t sign = (code >> (total_bits - 1)) & 1u;
    const uint32_t field_e = (code >> fs.mant_bits) & ((1u << fs.exp_bits) - 1u);
    const uint32_t field_m = code & ((1u << fs.mant_bits) - 1u);
    double a;
    const uint32_t e_all_ones = (1u << fs.exp_bits) - 1u;
    if (fmt == FMT_E4M3) {
        // E4M3 ("fn" flavour): no infinities, the single NaN is exponent and mantissa all ones
        if (field_e == e_all_ones && field_m == 7u) return std::nanf("");
    } else if (field_e == e_all_ones) {
        if (field_m != 0) return std::nanf("");
        return sign ? -INFINITY : INFINITY;
    }
    if (field_e == 0) a = std::ldexp((double)field_m, fs.e_min - fs.mant_bits);
    else a = std::ldexp(1.0 + std::ldexp((double)field_m, -fs.mant_bits), (int)field_e - fs.bias);
    return (float)(sign ? -a : a);
}

int code_bytes(int fmt) { return (fmt == FMT_E4M3 || is_int_format(fmt)) ? 1 : (fmt == FMT_FP32 ? 4 : 2); }

uint32_t load_code(const void* base, uint64_t i, int fmt) {
    switch (code_bytes(fmt)) {
        case 1: return ((const uint8_t*)base)[i];
        case 2: return ((const uint16_t*)base)[i];
        default: return ((const uint32_t*)base)[i];
    }
}
void store_code(void* base, uint64_t i, int fmt, uint32_t code) {
    switch (code_bytes(fmt)) {
        case 1: ((uint8_t*)base)[i] = (uint8_t)code; break;
        case 2: ((uint16_t*)base)[i] = (uint16_t)code; break;
        default: ((uint32_t*)base)[i] = code; break;
    }
}

// ------------------------------------------------------------------------------------------
// exp_spec: the decay a = exp(dt * A) must be the same binary32 number on every implementation,
// because any last-bit difference is fed back through the recurrence for the rest of the run.
// The paper only says exp(A * dt); this build fixes it as the following sequence of binary32
// operations: clamp, round z / ln2 to an integer k, two-constant Cody-Waite reduction with fmaf,
// degree-7 Taylor polynomial by Horner with fmaf, scale by 2^k.
// ------------------------------------------------------------------------------------------
float exp_spec(float z) {
    const float LOG2E = 0x1.715476p+0f;
    const float LN2_HI = 0x1.62e400p-1f;
    const float LN2_LO = 0x1.7f7d1cp-20f;
    if (!(z > -87.0f)) z = -87.0f;
    if (z > 88.0f) z = 88.0f;
    const float k = std::nearbyintf(z * LOG2E);  // ties to even
    float r = std::fmaf(k, -LN2_HI, z);
    r = std::fmaf(k, -LN2_LO, r);
    float p = 0x1.a01a02p-13f;          // 1/7!
    p = std::fmaf(p, r, 0x1.6c16c2p-10f);  // 1/6!
    p = std::fmaf(p, r, 0x1.111112p-7f);   // 1/5!
    p = std::fmaf(p, r, 0x1.555556p-5f);   // 1/4!
    p = std::fmaf(p, r, 0x1.555556p-3f);   // 1/3!
    p = std::fmaf(p, r, 0.5f);             // 1/2!
    p = std::fmaf(p, r, 1.0f);
    p = std::fmaf(p, r, 1.0f);
    return std::ldexp(p, (int)k);  // exact: the result is a normal number for z in [-87, 88]
}

// softplus_spec: dt = softplus(dt_raw + dt_bias) feeds the decay and the write term, so like exp_spec it has to be
// one fixed sequence of binary32 operations.  softplus(x) = max(x, 0) + log1p(exp(-|x|)), and for t in (0, 1]
// log1p(t) = 2 atanh(u) with u = t / (2 + t) <= 1/3: an odd series in u, cut after u^15 (relative 1e-9).  Above
// 20 the function returns x, the customary threshold of selective-state-update implementations.
float softplus_spec(float x) {
    if (x > 20.0f) return x;
    const float t = exp_spec(-std::fabs(x));
    const float u = t / (2.0f + t);
    const float s = u * u;
    float p = 0x1.111112p-3f;            // 2/15
    p = std::fmaf(p, s, 0x1.3b13b2p-3f); // 2/13
    p = std::fmaf(p, s, 0x1.745d18p-3f); // 2/11
    p = std::fmaf(p, s, 0x1.c71c72p-3f); // 2/9
    p = std::fmaf(p, s, 0x1.24924ap-2f); // 2/7
    p = std::fmaf(p, s, 0x1.99999ap-2f); // 2/5
    p = std::fmaf(p, s, 0x1.555556p-1f); // 2/3
    p = std::fmaf(p, s, 2.0f);
    return std::fmaf(u, p, std::max(x, 0.0f));
}

// Block scale of the E4M3 store: s = max|h'| / 448 in FP32 (Appendix B "Formats"), floored at the
// smallest normal number so that an all-zero block is well defined.  Entries are multiplied by
// 1/s, rounded once per block, instead of being divided by s one by one.
float block_scale(float amax, int fmt) {
    const float top = is_int_format(fmt) ? (float)int_qmax(fmt) : 448.0f;
    return std::max(amax / top, FLT_MIN);
}

}  // namespace

extern "C" {

// ---- elementary functions, exported so that each can be pinned on its own -------------------
uint32_t oracle_weyl_acc(uint32_t r, uint32_t c, uint32_t layer, uint32_t seed, uint32_t t) {
    return weyl_acc(r, c, layer, seed, t);
}
void oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) { philox4x32_10(ctr, key, out); }
float oracle_exp_spec(float z) { return exp_spec(z); }
uint32_t oracle_fmix32(uint32_t h) { return fmix32(h); }
float oracle_softplus_spec(float x) { return softplus_spec(x); }
// the block scale of a scaled store for an array of block maxima (exported so that it can be pinned on its own)
void oracle_block_scale_array(const float* amax, uint64_t n, int fmt, float* out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)n; ++i) out[i] = block_scale(amax[i], fmt);
}
void oracle_softplus_spec_array(const float* x, uint64_t n, float* out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)n; ++i) out[i] = softplus_spec(x[i]);
}
float oracle_round(float v, int fmt, int rule, uint32_t U) { return round_on_grid(v, fmt, rule, U); }
uint32_t oracle_encode(float q, int fmt) { return encode(q, fmt); }
float oracle_decode(uint32_t code, int fmt) { return decode(code, fmt); }
uint32_t oracle_threshold(int rule, uint32_t layer, uint32_t weyl_seed, uint32_t weyl_block, uint64_t sr_seed,
                          uint64_t flat, uint32_t t) {
    RuleParams rp{rule, layer, weyl_seed, weyl_block, sr_seed};
    return threshold_u24(rp, flat, t);
}
void oracle_round_array(const float* v, const uint32_t* U, uint64_t n, int fmt, int rule, float* out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)n; ++i) out[i] = round_on_grid(v[i], fmt, rule, U[i]);
}
// Eq. 2 and the encoding, entry by entry, with the thresholds given: codes[i] = encode(round(v[i]; U[i])).
// U may be null (RTN), or hold one value used for every entry (n_U == 1).
void oracle_round_encode_array(const float* v, const uint32_t* U, uint64_t n_U, uint64_t n, int fmt, int rule, void* codes) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)n; ++i) {
        const uint32_t u = U ? U[n_U == 1 ? 0 : i] : 0u;
        store_code(codes, (uint64_t)i, fmt, encode(round_on_grid(v[i], fmt, rule, u), fmt));
    }
}
void oracle_exp_spec_array(const float* z, uint64_t n, float* out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)n; ++i) out[i] = exp_spec(z[i]);
}

// ---- one decode step of one layer (Eq. 1 + readout + Eq. 2), in place -----------------------
// state  : [B, H, P, N] codes of `fmt` (FMT_FP32: floats, no rounding = the fp32-state twin)
// scales : E4M3 only, [B, H, P, N / scale_block] floats, or [B, H] when scale_block == P * N
// x [B,H,P], dt [B,H], A [H] or [H,N] (a_per_state), Bm, Cm [B,G,N], D [H] or null, y [B,H,P]
// The rest of a production selective-state-update signature (Appendix B "Runners" keeps the grouped B and C and the
// output gate of the Mamba implementations it follows): dt_bias [H] or null, dt_softplus (dt <- softplus_spec(dt + dt_bias)), ngroups G
// (head h reads group h / (H / G)), z [B,H,P] or null (y <- y * z * sigmoid(z)).
// head_index_base, nheads_global: the call holds heads head_index_base .. head_index_base + H - 1 of a layer with
// nheads_global heads (0 = H); like batch_index_base they only enter the entry index that the thresholds are drawn from.
// Returns 0, or -1 on an argument the oracle does not define.
int oracle_state_update(void* state, float* scales, int fmt, uint32_t scale_block,
                        uint32_t B, uint32_t H, uint32_t P, uint32_t N,
                        const float* x, const float* dt, const float* A, int a_per_state,
                        const float* Bm, const float* Cm, const float* D, float* y,
                        int rule, uint32_t layer, uint32_t weyl_seed, uint32_t weyl_block, uint64_t sr_seed,
                        uint32_t batch_index_base, uint32_t step_t,
                        const float* dt_bias, int dt_softplus, uint32_t ngroups, const float* z,
                        uint32_t head_index_base, uint32_t nheads_global) {
    if (ngroups == 0) ngroups = 1;
    if (nheads_global == 0) nheads_global = H;
    if (head_index_base + H > nheads_global) return -1;
    if (H % ngroups != 0) return -1;
    const uint32_t heads_per_group = H / ngroups;
    if (has_block_scale(fmt)) {
        if (scale_block == 0 || !scales) return -1;
        if (!(scale_block == P * N || N % scale_block == 0)) return -1;
    }
    if (rule == RULE_WEYL && (weyl_block == 0 || N % weyl_block != 0)) return -1;
    const RuleParams rp{rule, layer, weyl_seed, weyl_block, sr_seed};
    const bool head_scale = (has_block_scale(fmt) && scale_block == P * N && scale_block != N);
    const int64_t BH = (int64_t)B * H;
#pragma omp parallel for schedule(static)
    for (int64_t bh = 0; bh < BH; ++bh) {
        const uint32_t b = (uint32_t)(bh / H), h = (uint32_t)(bh % H);
        float dtv = dt[bh];
        if (dt_bias) dtv = dtv + dt_bias[h];
        if (dt_softplus) dtv = softplus_spec(dtv);
        const float* Bg = Bm + ((uint64_t)b * ngroups + h / heads_per_group) * N;
        const float* Cg = Cm + ((uint64_t)b * ngroups + h / heads_per_group) * N;
        std::vector<float> hp((size_t)P * N);
        // Eq. 1 in FP32: a = exp(dt*A), w = (dt*x)*B, h' = fma(a, h, w); dequantise first.
        for (uint32_t p = 0; p < P; ++p) {
            const float xv = x[(uint64_t)bh * P + p];
            const float dtx = dtv * xv;
            for (uint32_t n = 0; n < N; ++n) {
                const uint64_t local = ((uint64_t)bh * P + p) * N + n;
                float hv = decode(load_code(state, local, fmt), fmt);
                if (has_block_scale(fmt)) {
                    const uint64_t sidx = head_scale ? (uint64_t)bh : local / scale_block;
                    hv = hv * scales[sidx];
                }
                const float Av = a_per_state ? A[(uint64_t)h * N + n] : A[h];
                const float a = exp_spec(dtv * Av);
                const float w = dtx * Bg[n];
                hp[(size_t)p * N + n] = std::fmaf(a, hv, w);
            }
            // readout from the unrounded h', accumulated in double and rounded once
            double acc = 0.0;
            for (uint32_t n = 0; n < N; ++n) acc += (double)Cg[n] * (double)hp[(size_t)p * N + n];
            if (D) acc += (double)D[h] * (double)xv;
            if (z) {
                const double zv = (double)z[(uint64_t)bh * P + p];
                acc *= zv / (1.0 + std::exp(-zv));
            }
            y[(uint64_t)bh * P + p] = (float)acc;
        }
        // write-back: block scale (E4M3), threshold, Eq. 2, encode
        const uint64_t head_elems = (uint64_t)P * N;
        const uint64_t blk = has_block_scale(fmt) ? scale_block : head_elems;
        for (uint64_t s0 = 0; s0 < head_elems; s0 += blk) {
            float rinv = 1.0f;
            if (has_block_scale(fmt)) {
                float amax = 0.0f;
                for (uint64_t i = s0; i < s0 + blk; ++i) amax = std::max(amax, std::fabs(hp[i]));
                const float s = block_scale(amax, fmt);
                rinv = 1.0f / s;
                scales[((uint64_t)bh * head_elems + s0) / blk] = s;
            }
            for (uint64_t i = s0; i < s0 + blk; ++i) {
                const uint64_t local = (uint64_t)bh * head_elems + i;
                // the index of the entry in the whole layer, of which this call may hold a slice of the batch and of the heads
                const uint64_t flat = (((uint64_t)batch_index_base + b) * nheads_global + head_index_base + h) * head_elems + i;
                const float v = has_block_scale(fmt) ? hp[i] * rinv : hp[i];
                const uint32_t U = threshold_u24(rp, flat, step_t);
                store_code(state, local, fmt, encode(round_on_grid(v, fmt, rule, U), fmt));
            }
        }
    }
    return 0;
}

// ---- quantise an FP32 array into a store (used to seed h_0 from a full-precision state) ------
// src [n_rows, row_len]; scale blocks lie along the row (row_len % scale_block == 0).
int oracle_quantize_store(const float* src, void* dst_codes, float* dst_scales, uint64_t n_rows, uint32_t row_len,
                          int fmt, uint32_t scale_block, int rule, uint32_t layer, uint32_t weyl_seed,
                          uint32_t weyl_block, uint64_t sr_seed, uint64_t row_index_base, uint32_t step_t) {
    if (has_block_scale(fmt) && (scale_block == 0 || row_len % scale_block != 0 || !dst_scales)) return -1;
    if (rule == RULE_WEYL && (weyl_block == 0 || row_len % weyl_block != 0)) return -1;
    const RuleParams rp{rule, layer, weyl_seed, weyl_block, sr_seed};
    const uint32_t blk = has_block_scale(fmt) ? scale_block : row_len;
#pragma omp parallel for schedule(static)
    for (int64_t row = 0; row < (int64_t)n_rows; ++row) {
        for (uint32_t s0 = 0; s0 < row_len; s0 += blk) {
            float rinv = 1.0f;
            if (has_block_scale(fmt)) {
                float amax = 0.0f;
                for (uint32_t i = s0; i < s0 + blk; ++i) amax = std::max(amax, std::fabs(src[(uint64_t)row * row_len + i]));
                const float s = block_scale(amax, fmt);
                rinv = 1.0f / s;
                dst_scales[((uint64_t)row * row_len + s0) / blk] = s;
            }
            for (uint32_t i = s0; i < s0 + blk; ++i) {
                const uint64_t local = (uint64_t)row * row_len + i;
                const uint64_t flat = row_index_base * row_len + local;
                const float h = src[local];
                const float v = has_block_scale(fmt) ? h * rinv : h;
                const uint32_t U = threshold_u24(rp, flat, step_t);
                store_code(dst_codes, local, fmt, encode(round_on_grid(v, fmt, rule, U), fmt));
            }
        }
    }
    return 0;
}

// ---- open-loop replay of recorded traces (Appendix B "Open-loop replay"): h_t = Q(a_t h_{t-1} + w_t) ------
// codes [n_rows, row_len] (and scales) are updated in place from w [n_rows, row_len] and one decay per
// `rows_per_decay` consecutive rows (a [n_rows / rows_per_decay]; a head of P rows shares its decay).  FP32:
// h' = fma(a, dequant(code), w); then block scale, threshold and Eq. 2 exactly as in the decode step.
int oracle_replay_step(const float* w, const float* a, uint32_t rows_per_decay, void* codes, float* scales,
                       uint64_t n_rows, uint32_t row_len, int fmt, uint32_t scale_block, int rule, uint32_t layer,
                       uint32_t weyl_seed, uint32_t weyl_block, uint64_t sr_seed, uint64_t row_index_base, uint32_t step_t) {
    if (has_block_scale(fmt) && (scale_block == 0 || row_len % scale_block != 0 || !scales)) return -1;
    if (rule == RULE_WEYL && (weyl_block == 0 || row_len % weyl_block != 0)) return -1;
    if (rows_per_decay == 0 || n_rows % rows_per_decay != 0) return -1;
    const RuleParams rp{rule, layer, weyl_seed, weyl_block, sr_seed};
    const uint32_t blk = has_block_scale(fmt) ? scale_block : row_len;
#pragma omp parallel for schedule(static)
    for (int64_t row = 0; row < (int64_t)n_rows; ++row) {
        const float av = a[row / rows_per_decay];
        std::vector<float> hp(row_len);
        for (uint32_t i = 0; i < row_len; ++i) {
            const uint64_t local = (uint64_t)row * row_len + i;
            float hv = decode(load_code(codes, local, fmt), fmt);
            if (has_block_scale(fmt)) hv = hv * scales[local / scale_block];
            hp[i] = std::fmaf(av, hv, w[local]);
        }
        for (uint32_t s0 = 0; s0 < row_len; s0 += blk) {
            float rinv = 1.0f;
            if (has_block_scale(fmt)) {
                float amax = 0.0f;
                for (uint32_t i = s0; i < s0 + blk; ++i) amax = std::max(amax, std::fabs(hp[i]));
                const float s = block_scale(amax, fmt);
                rinv = 1.0f / s;
                scales[((uint64_t)row * row_len + s0) / blk] = s;
            }
            for (uint32_t i = s0; i < s0 + blk; ++i) {
                const uint64_t local = (uint64_t)row * row_len + i;
                const uint64_t flat = row_index_base * row_len + local;
                const float v = has_block_scale(fmt) ? hp[i] * rinv : hp[i];
                const uint32_t U = threshold_u24(rp, flat, step_t);
                store_code(codes, local, fmt, encode(round_on_grid(v, fmt, rule, U), fmt));
            }
        }
    }
    return 0;
}

// Dequantise a store back to FP32 (for error metrics and for reading results).
void oracle_dequantize(const void* codes, const float* scales, uint64_t n, int fmt, uint32_t scale_block, float* out) {
    for (uint64_t i = 0; i < n; ++i) {
        float v = decode(load_code(codes, i, fmt), fmt);
        if (has_block_scale(fmt)) v = v * scales[i / scale_block];
        out[i] = v;
    }
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    int n = 1;
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
    return n;
#else
    return 1;
#endif
}

}  // extern "C"

// ssdq_quantize.cu -- stand-alone use of the rounding functions: quantise an FP32 array into a store
// (Eq. 2 under the chosen rule), dequantise a store, and materialise thresholds for inspection.
#include "ssdq_update.cuh"

namespace ssdq {

// One slot (LPR lanes) per row, grid-stride over rows; same lane-to-entry mapping as the fused kernel.
// REPLAY: the open-loop replay step h <- Q(a h + src) (Appendix B "Open-loop replay"): the old codes are
// dequantised, multiplied by the row's recorded decay and the recorded write is added with one fused multiply-add.
template <int FMT, int RULE, int LPR, bool REPLAY>
__global__ void __launch_bounds__(kThreads) quantize_kernel(const QuantParams p) {
    constexpr int EPL = Fmt<FMT>::kEpl;
    constexpr int N = LPR * EPL;
    constexpr unsigned FULL = 0xFFFFFFFFu;
    constexpr uint32_t NSLOT = kThreads / LPR;
    const uint32_t lis = threadIdx.x % LPR;
    const uint32_t slot = threadIdx.x / LPR;
    LaneThreshold<FMT, RULE, LPR> thr;
    thr.init(p.weyl, p.step_t, lis);
    const uint32_t key0 = (uint32_t)p.sr_seed, key1 = (uint32_t)(p.sr_seed >> 32);
    const bool row_scale = Fmt<FMT>::kScaled && (p.scale_block == (uint32_t)N);
    const uint64_t rows_per_pass = (uint64_t)gridDim.x * NSLOT;
    const uint64_t n_pass = (p.n_rows + rows_per_pass - 1) / rows_per_pass;    // uniform trip count: shuffles inside
    for (uint64_t it = 0; it < n_pass; ++it) {
        const uint64_t row = it * rows_per_pass + (uint64_t)blockIdx.x * NSLOT + slot;
        const bool ok = row < p.n_rows;
        float v[EPL];
#pragma unroll
        for (int i = 0; i < EPL / 4; ++i) {
            float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
            if (ok) f = reinterpret_cast<const float4*>(p.src + row * N + lis * EPL)[i];
            v[4 * i] = f.x; v[4 * i + 1] = f.y; v[4 * i + 2] = f.z; v[4 * i + 3] = f.w;
        }
        if constexpr (REPLAY) {
            float h[EPL];
            uint4 raw = make_uint4(0u, 0u, 0u, 0u);
            float a = 0.0f, s_old = 0.0f;
            if (ok) {
                raw = reinterpret_cast<const uint4*>(p.codes)[row * LPR + lis];
                a = __ldg(p.decay + row / p.rows_per_decay);
                if constexpr (Fmt<FMT>::kScaled) s_old = row_scale ? p.scales[row] : p.scales[row * (N / 16) + lis];
            }
            unpack_lane<FMT>(raw, h);
#pragma unroll
            for (int j = 0; j < EPL; ++j) {
                float hin = h[j];
                if constexpr (Fmt<FMT>::kScaled) hin = __fmul_rn(hin, s_old);
                v[j] = __fmaf_rn(a, hin, v[j]);
            }
        }
        if constexpr (Fmt<FMT>::kScaled) {
            float amax = 0.0f;
#pragma unroll
            for (int j = 0; j < EPL; ++j) amax = fmaxf(amax, fabsf(v[j]));
            if (row_scale) {
#pragma unroll
                for (int off = LPR / 2; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, off));
            }
            const float s = fmaxf(__fdiv_rn(amax, p.scale_top), 1.17549435e-38f);
            const float rinv = __frcp_rn(s);
#pragma unroll
            for (int j = 0; j < EPL; ++j) v[j] = __fmul_rn(v[j], rinv);
            if (ok) {
                if (row_scale) { if (lis == 0) p.scales[row] = s; }
                else p.scales[row * (N / 16) + lis] = s;
            }
        }
        const uint64_t grow = p.row_base + row + (p.rows_per_seq ? (row / p.rows_per_seq) * p.row_skip : 0ull);
        uint32_t g_lo = 0, g_hi = 0, acc0 = 0;
        if constexpr (RULE == RULE_WEYL) acc0 = thr.weyl_acc0(grow);
        if constexpr (RULE == RULE_SR_HASH) acc0 = thr.hash_key0(grow, p.step_t * kHashP2 + p.layer * kHashP3 + key0 * kHashP4, key1);
        if constexpr (RULE == RULE_SR) thr.sr_group(grow, g_lo, g_hi);
        const uint4 packed = round_pack_lane<FMT, RULE>(v, acc0, p.weyl.mul_col, g_lo, g_hi, p.step_t, p.layer, key0, key1, p.scale_top);
        if (ok) reinterpret_cast<uint4*>(p.codes)[row * LPR + lis] = packed;
    }
}

template <int FMT, int RULE, int LPR>
static cudaError_t launch_quantize_one(const QuantParams& p, cudaStream_t s) {
    constexpr uint32_t NSLOT = kThreads / LPR;
    uint64_t grid = (p.n_rows + NSLOT - 1) / NSLOT;
    if (grid > 148u * 64u) grid = 148u * 64u;
    if (grid == 0) return cudaSuccess;
    if (p.decay) quantize_kernel<FMT, RULE, LPR, true><<<(unsigned)grid, kThreads, 0, s>>>(p);
    else quantize_kernel<FMT, RULE, LPR, false><<<(unsigned)grid, kThreads, 0, s>>>(p);
    return cudaGetLastError();
}

template <int FMT, int RULE>
static cudaError_t launch_quantize_n(const QuantParams& p, cudaStream_t s) {
    constexpr int EPL = Fmt<FMT>::kEpl;
    if (p.row_len % EPL != 0) return cudaErrorInvalidValue;
    switch (p.row_len / EPL) {
        case 1: if constexpr (EPL == 16) return launch_quantize_one<FMT, RULE, 1>(p, s); break;
        case 2: if constexpr (EPL >= 8) return launch_quantize_one<FMT, RULE, 2>(p, s); break;
        case 4: return launch_quantize_one<FMT, RULE, 4>(p, s);
        case 8: return launch_quantize_one<FMT, RULE, 8>(p, s);
        case 16: return launch_quantize_one<FMT, RULE, 16>(p, s);
        case 32: if constexpr (EPL <= 8) return launch_quantize_one<FMT, RULE, 32>(p, s); break;
        default: break;
    }
    return cudaErrorInvalidValue;
}

template <int FMT>
static cudaError_t launch_quantize_fmt(const QuantParams& p, int rule, cudaStream_t s) {
    switch (rule) {
        case RULE_RTN: return launch_quantize_n<FMT, RULE_RTN>(p, s);
        case RULE_SR: return launch_quantize_n<FMT, RULE_SR>(p, s);
        case RULE_WEYL: return launch_quantize_n<FMT, RULE_WEYL>(p, s);
        case RULE_SR_HASH: return launch_quantize_n<FMT, RULE_SR_HASH>(p, s);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_quantize(const QuantParams& p, int fmt, int rule, cudaStream_t s) {
    switch (fmt) {
        case FMT_FP16: return launch_quantize_fmt<FMT_FP16>(p, rule, s);
        case FMT_BF16: return launch_quantize_fmt<FMT_BF16>(p, rule, s);
        case FMT_E4M3: return launch_quantize_fmt<FMT_E4M3>(p, rule, s);
        case FMT_INT: return launch_quantize_fmt<FMT_INT>(p, rule, s);
        case FMT_FP32: return launch_quantize_n<FMT_FP32, RULE_RTN>(p, s);
        default: return cudaErrorInvalidValue;
    }
}

// ---- dequantise: one lane per 16 bytes of codes ------------------------------------------------
template <int FMT>
__global__ void __launch_bounds__(256) dequantize_kernel(const uint4* __restrict__ codes, const float* __restrict__ scales,
                                                         uint64_t n_vec, uint32_t scale_block, float* __restrict__ out) {
    constexpr int EPL = Fmt<FMT>::kEpl;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += (uint64_t)gridDim.x * blockDim.x) {
        float h[EPL];
        unpack_lane<FMT>(codes[i], h);
        if constexpr (Fmt<FMT>::kScaled) {
            const float s = scales[(i * EPL) / scale_block];     // 16 consecutive entries share a scale
#pragma unroll
            for (int j = 0; j < EPL; ++j) h[j] = __fmul_rn(h[j], s);
        }
#pragma unroll
        for (int j = 0; j < EPL / 4; ++j)
            reinterpret_cast<float4*>(out + i * EPL)[j] = make_float4(h[4 * j], h[4 * j + 1], h[4 * j + 2], h[4 * j + 3]);
    }
}

cudaError_t launch_dequantize(const void* codes, const float* scales, uint64_t n, int fmt, uint32_t scale_block,
                              float* out, cudaStream_t s) {
    if (n == 0) return cudaSuccess;
    const uint4* c = reinterpret_cast<const uint4*>(codes);
    auto grid_of = [](uint64_t n_vec) { uint64_t g = (n_vec + 255) / 256; return (unsigned)(g > 148u * 32u ? 148u * 32u : g); };
    switch (fmt) {
        case FMT_FP16: dequantize_kernel<FMT_FP16><<<grid_of(n / 8), 256, 0, s>>>(c, scales, n / 8, scale_block, out); break;
        case FMT_BF16: dequantize_kernel<FMT_BF16><<<grid_of(n / 8), 256, 0, s>>>(c, scales, n / 8, scale_block, out); break;
        case FMT_E4M3: dequantize_kernel<FMT_E4M3><<<grid_of(n / 16), 256, 0, s>>>(c, scales, n / 16, scale_block, out); break;
        case FMT_INT: dequantize_kernel<FMT_INT><<<grid_of(n / 16), 256, 0, s>>>(c, scales, n / 16, scale_block, out); break;
        case FMT_FP32: dequantize_kernel<FMT_FP32><<<grid_of(n / 4), 256, 0, s>>>(c, scales, n / 4, scale_block, out); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

// ---- thresholds, one thread per entry, straight from the definitions ---------------------------
__global__ void __launch_bounds__(256) thresholds_kernel(int rule, WeylConst w, uint64_t sr_seed, uint32_t layer,
                                                         uint64_t first_flat, uint64_t n, uint32_t step_t,
                                                         uint32_t* __restrict__ out) {
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t flat = first_flat + i;
        uint32_t U = 0;
        if (rule == RULE_WEYL) {
            const uint32_t r = (uint32_t)(flat / w.block), c = (uint32_t)(flat % w.block);
            U = (w.mul_row * (r + 1u) + w.mul_col * (c + 1u) + w.base + step_t * w.phi) >> 8;
        } else if (rule == RULE_SR) {
            const uint64_t g = flat >> 2;
            const uint4 o = philox4x32_10(make_uint4((uint32_t)g, (uint32_t)(g >> 32), step_t, layer),
                                          (uint32_t)sr_seed, (uint32_t)(sr_seed >> 32));
            const uint32_t word[4] = {o.x, o.y, o.z, o.w};
            U = word[flat & 3u] >> 8;
        } else if (rule == RULE_SR_HASH) {
            const uint32_t key = (uint32_t)flat * kHashP1 + step_t * kHashP2 + layer * kHashP3 + (uint32_t)sr_seed * kHashP4 +
                                 ((uint32_t)(flat >> 32) ^ (uint32_t)(sr_seed >> 32)) * kHashP5;
            U = fmix32(key) >> 8;
        }
        out[i] = U;
    }
}

cudaError_t launch_thresholds(int rule, const WeylConst& w, uint64_t sr_seed, uint32_t layer, uint64_t first_flat,
                              uint64_t n, uint32_t step_t, uint32_t* out, cudaStream_t s) {
    if (n == 0) return cudaSuccess;
    uint64_t g = (n + 255) / 256;
    if (g > 148u * 32u) g = 148u * 32u;
    thresholds_kernel<<<(unsigned)g, 256, 0, s>>>(rule, w, sr_seed, layer, first_flat, n, step_t, out);
    return cudaGetLastError();
}

}  // namespace ssdq

// ssdq_update.cuh -- the fused decode-step kernel: dequantise -> Eq. 1 -> readout -> threshold ->
// Eq. 2 -> encode -> store, one pass over the state, bounded by HBM bandwidth.
//
// Data layout and thread mapping.  The state is [B, H, P, N] with N contiguous; a row (b, h, p) is
// N codes.  Each lane owns 16 bytes of a row (EPL = 8 two-byte codes, 16 E4M3 codes or 4 floats), so a
// row is held by LPR = N / EPL neighbouring lanes (a "slot").  A CTA of kThreads lanes has
// kThreads / LPR slots; they are split over `items_per_cta` (b, h) items, `spi` slots per item, and a
// slot walks `rps` consecutive rows p of its item.  A lane therefore keeps its B[n], C[n] (and its
// decays when A is per state) in registers for the whole CTA, issues UNR independent 128-bit loads
// before it touches the first of them, and produces one partial dot per row which the slot reduces
// with xor-shuffles.  Nothing is shared between CTAs, every state byte has one reader-then-writer.
#pragma once
#include "ssdq_device.cuh"
#include "ssdq_internal.h"

namespace ssdq {

constexpr int kThreads = 128;

template <int FMT> struct Unroll { static constexpr int value = 4; };
template <> struct Unroll<FMT_E4M3> { static constexpr int value = 2; };
template <> struct Unroll<FMT_INT> { static constexpr int value = 2; };

// Unpack the lane's 16 bytes into EPL floats (exact widening; E4M3 is multiplied by its scale later).
template <int FMT>
__device__ __forceinline__ void unpack_lane(const uint4& raw, float* h) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    if constexpr (FMT == FMT_FP16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack2_fp16(w[i], h[2 * i], h[2 * i + 1]);
    } else if constexpr (FMT == FMT_BF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack2_bf16(w[i], h[2 * i], h[2 * i + 1]);
    } else if constexpr (FMT == FMT_E4M3) {
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack4_e4m3(w[i], h + 4 * i);
    } else if constexpr (FMT == FMT_INT) {
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack4_int8(w[i], h + 4 * i);
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) h[i] = __uint_as_float(w[i]);
    }
}

// Round the lane's EPL values v[] under RULE and pack them into 16 bytes.
// acc0: Weyl accumulator of the lane's first entry (RULE_WEYL); ctr/key: Philox counter of the
// lane's first group of four entries (RULE_SR).
template <int FMT, int RULE>
__device__ __forceinline__ uint4 round_pack_lane(const float* v, uint32_t acc0, uint32_t mul_col, uint32_t g_lo,
                                                 uint32_t g_hi, uint32_t step_t, uint32_t layer, uint32_t key0,
                                                 uint32_t key1, float qmax) {
    constexpr int EPL = Fmt<FMT>::kEpl;
    uint32_t w[4] = {0u, 0u, 0u, 0u};       // (every path below sets all four; the one-byte formats return early)
    if constexpr (FMT == FMT_FP32) {
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = __float_as_uint(v[i]);
    } else if constexpr (RULE == RULE_RTN) {
        if constexpr (FMT == FMT_FP16) {
#pragma unroll
            for (int i = 0; i < 4; ++i) w[i] = rtn_pack2_fp16(v[2 * i], v[2 * i + 1]);
        } else if constexpr (FMT == FMT_BF16) {
#pragma unroll
            for (int i = 0; i < 4; ++i) w[i] = rtn_pack2_bf16(v[2 * i], v[2 * i + 1]);
        } else {
            return round_pack16<FMT, RULE_RTN>(v, nullptr, qmax);
        }
    } else {
        uint32_t acc[EPL];
        if constexpr (RULE == RULE_WEYL) {
#pragma unroll
            for (int k = 0; k < EPL; ++k) acc[k] = acc0 + (uint32_t)k * mul_col;
        } else if constexpr (RULE == RULE_SR_HASH) {
#pragma unroll
            for (int k = 0; k < EPL; ++k) acc[k] = fmix32(acc0 + (uint32_t)k * kHashP1);    // acc0 = hash key of the first entry
        } else {
#pragma unroll
            for (int g = 0; g < EPL / 4; ++g) {
                const uint32_t lo = g_lo + (uint32_t)g;           // g_lo is a multiple of EPL / 4: no carry
                const uint4 o = philox4x32_10(make_uint4(lo, g_hi, step_t, layer), key0, key1);
                acc[4 * g] = o.x; acc[4 * g + 1] = o.y; acc[4 * g + 2] = o.z; acc[4 * g + 3] = o.w;
            }
        }
        // BF16 and FP16: the hardware stochastic-rounding converts.  Both take, per input, the leading bits of
        // (threshold XOR sign mask): a negative value takes ~U.
        if constexpr (FMT == FMT_BF16) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t b0 = __float_as_uint(v[2 * i]), b1 = __float_as_uint(v[2 * i + 1]);
                const uint32_t x0 = acc[2 * i] ^ (uint32_t)((int32_t)b0 >> 31);
                const uint32_t x1 = acc[2 * i + 1] ^ (uint32_t)((int32_t)b1 >> 31);
                w[i] = sr_pack2_bf16_fields(v[2 * i], v[2 * i + 1], __byte_perm(x0, x1, 0x7632));     // the top halves
            }
        } else if constexpr (FMT == FMT_FP16) {
            float vmin0 = 3.0e38f, vmin1 = 3.0e38f;
            uint32_t f[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                // the two fields of a pair at once: the top halves of the two accumulators, XOR the two sign bytes
                // replicated over their halves
                const uint32_t tops = __byte_perm(acc[2 * i], acc[2 * i + 1], 0x7632);
                const uint32_t signs = sign_halves(v[2 * i], v[2 * i + 1]);
                f[i] = (tops ^ signs) >> 3;        // the leading 13 bits of each in [12:0] and [28:16]; the convert ignores bits [15:13]
                if (i & 1) vmin1 = min3abs(vmin1, v[2 * i], v[2 * i + 1]);
                else vmin0 = min3abs(vmin0, v[2 * i], v[2 * i + 1]);
            }
            if (fminf(vmin0, vmin1) >= 0x1p-14f) {
                // every target is in FP16's normal range: the 13 dropped bits are all carried by the field, one convert is exact
#pragma unroll
                for (int i = 0; i < 4; ++i) w[i] = sr_pack2_fp16(v[2 * i], v[2 * i + 1], f[i]);
            } else {
                // below 2^-14 the threshold has more leading bits than the field carries: fields f and f + 1 bracket the
                // true addend, and where the two codes differ (or f + 1 does not fit) the lane decides exactly
                uint32_t unsure = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t f1 = (f[i] & 0x1FFF1FFFu) + 0x00010001u;
                    w[i] = sr_pack2_fp16(v[2 * i], v[2 * i + 1], f[i]);
                    unsure |= (w[i] ^ sr_pack2_fp16(v[2 * i], v[2 * i + 1], f1)) | (f1 & 0x20002000u);
                }
                if (unsure) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float r[2];
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const float vv = v[2 * i + j];
                            const float scale = dither_step_scale<10, -14, 24>(vv);
                            const float q = floor_to_step(dithered_sum_rm(vv, acc[2 * i + j], scale), scale);
                            // sign of v forced onto the result (it already has it unless it is zero)
                            r[j] = __uint_as_float((__float_as_uint(q) & 0x7FFFFFFFu) | (__float_as_uint(vv) & 0x80000000u));
                        }
                        w[i] = rtn_pack2_fp16(r[0], r[1]);   // exact: r is on the FP16 grid; saturates beyond 65504
                    }
                }
            }
        } else {
            return round_pack16<FMT, RULE>(v, acc, qmax);
        }
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Asynchronous global -> shared copies (cg: through L2 only; ca: also kept in L1), grouped by commit.
__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async16_ca(uint32_t smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async4_ca(uint32_t smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }

// Programmatic dependent launch.  Every fused-update kernel opens with grid_dependency_gate(): it waits until every
// earlier grid of the stream has completed and its writes are visible -- before the kernel touches any memory -- and
// lets the next kernel of the stream be scheduled, so that kernel's launch latency and CTA ramp overlap this one's
// execution.  The data dependency between the steps of a layer is kept by the wait (each kernel waits for its
// predecessor, which waited for its own, so completion is transitive).  Order of the two: a grid of many waves releases
// its successor first (the successor's CTAs can only become resident in the last wave anyway, and they are then in place
// when the tail drains); a small grid waits first, because releasing first lets waiting CTAs of several later launches
// pile up beside the running ones, which was measured to slow small launches down.  Launched without the attribute the
// two instructions do nothing.
__device__ __forceinline__ void grid_dependency_gate(uint32_t mode) {
    if (mode == 2u) asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (mode != 2u) asm volatile("griddepcontrol.launch_dependents;");
}

// One launch of a fused-update kernel; p.overlap adds the programmatic-stream-serialization attribute.
template <typename P>
inline cudaError_t launch_update_kernel(void (*kernel)(P), dim3 grid, size_t smem, cudaStream_t stream, const UpdateParams& p) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.overlap ? 1u : 0u;
    UpdateParams q = p;
    if (q.overlap && (uint64_t)grid.x * grid.y >= 1024u) q.overlap = 2u;     // several waves: release the successor first
    return cudaLaunchKernelEx(&cfg, kernel, q);
}

// Per-lane threshold set-up for the row with global index `grow` (row of the [B_global*H*P, N] view).
template <int FMT, int RULE, int LPR>
struct LaneThreshold {
    static constexpr int EPL = Fmt<FMT>::kEpl;
    static constexpr int N = LPR * EPL;
    uint32_t lane_const;   // Weyl: everything but the row term
    uint32_t row_mul;      // Weyl: mul_row * (dither blocks per row)
    uint32_t n0;

    __device__ __forceinline__ void init(const WeylConst& wc, uint32_t step_t, uint32_t lane_in_slot) {
        n0 = lane_in_slot * EPL;
        if constexpr (RULE == RULE_WEYL) {
            // block == N: r = grow, c = n;   block == 16: r = grow * (N/16) + n / 16, c = n % 16
            const bool row_block = (wc.block == (uint32_t)N);
            const uint32_t blocks_per_row = row_block ? 1u : (uint32_t)N / 16u;
            const uint32_t r_in_row = row_block ? 0u : n0 / 16u;
            const uint32_t c0 = row_block ? n0 : n0 % 16u;
            row_mul = wc.mul_row * blocks_per_row;
            lane_const = wc.mul_row * (r_in_row + 1u) + wc.mul_col * (c0 + 1u) + wc.base + step_t * wc.phi;
        }
    }
    __device__ __forceinline__ uint32_t weyl_acc0(uint64_t grow) const { return lane_const + row_mul * (uint32_t)grow; }
    // hash SR: key of the lane's first entry in row `grow`; hash_base = t*P2 + layer*P3 + seed_lo*P4
    __device__ __forceinline__ uint32_t hash_key0(uint64_t grow, uint32_t hash_base, uint32_t seed_hi) const {
        const uint64_t flat = grow * (uint64_t)N + n0;
        return (uint32_t)flat * kHashP1 + ((uint32_t)(flat >> 32) ^ seed_hi) * kHashP5 + hash_base;
    }
    __device__ __forceinline__ void sr_group(uint64_t grow, uint32_t& g_lo, uint32_t& g_hi) const {
        const uint64_t g = (grow * (uint64_t)N + n0) >> 2;
        g_lo = (uint32_t)g;
        g_hi = (uint32_t)(g >> 32);
    }
};

template <int FMT, int RULE, int LPR, bool APS>
__global__ void __launch_bounds__(kThreads) ssd_update_kernel(const UpdateParams p) {
    grid_dependency_gate(p.overlap);
    constexpr int EPL = Fmt<FMT>::kEpl;
    constexpr int N = LPR * EPL;
    constexpr int UNR = Unroll<FMT>::value;
    constexpr unsigned FULL = 0xFFFFFFFFu;

    const uint32_t step_t = p.step_t + (p.step_base ? __ldcg(p.step_base) : 0u);
    const uint32_t tid = threadIdx.x;
    const uint32_t lis = tid % LPR;                 // lane in slot
    const uint32_t slot = tid / LPR;
    const uint32_t item_raw = blockIdx.x * p.items_per_cta + slot / p.spi;
    const uint32_t sub = slot % p.spi;
    const bool item_ok = item_raw < p.n_items;
    const uint32_t item = item_ok ? item_raw : p.n_items - 1u;   // clamp: idle lanes still shuffle
    const uint32_t b = item / p.H;
    const uint32_t h = item - b * p.H;
    const uint32_t n0 = lis * EPL;

    // lane constants: B[n], C[n], decay(s), dt, D
    float Bv[EPL], Cv[EPL];
    {
        const size_t grp = (size_t)b * p.ngroups + h / p.heads_per_group;
        (void)SSDQ_RANGE_OK(p, DBG_BC, grp * N + n0, EPL, bc_floats);
        (void)SSDQ_RANGE_OK(p, DBG_ITEMS, item, 1, items);
        const float4* Bp = reinterpret_cast<const float4*>(p.Bm + grp * N + n0);
        const float4* Cp = reinterpret_cast<const float4*>(p.Cm + grp * N + n0);
#pragma unroll
        for (int i = 0; i < EPL / 4; ++i) {
            const float4 bb = __ldg(Bp + i), cc = __ldg(Cp + i);
            Bv[4 * i] = bb.x; Bv[4 * i + 1] = bb.y; Bv[4 * i + 2] = bb.z; Bv[4 * i + 3] = bb.w;
            Cv[4 * i] = cc.x; Cv[4 * i + 1] = cc.y; Cv[4 * i + 2] = cc.z; Cv[4 * i + 3] = cc.w;
        }
    }
    float dtv = __ldg(p.dt + item);
    if (p.dt_bias) dtv = __fadd_rn(dtv, __ldg(p.dt_bias + h));
    if (p.dt_softplus) dtv = softplus_spec(dtv);
    const float Dv = p.D ? __ldg(p.D + h) : 0.0f;
    float av[APS ? EPL : 1];
    if constexpr (APS) {
        const float4* Ap = reinterpret_cast<const float4*>(p.A + (size_t)h * N + n0);
#pragma unroll
        for (int i = 0; i < EPL / 4; ++i) {
            const float4 aa = __ldg(Ap + i);
            av[4 * i] = exp_spec(__fmul_rn(dtv, aa.x));
            av[4 * i + 1] = exp_spec(__fmul_rn(dtv, aa.y));
            av[4 * i + 2] = exp_spec(__fmul_rn(dtv, aa.z));
            av[4 * i + 3] = exp_spec(__fmul_rn(dtv, aa.w));
        }
    } else {
        av[0] = exp_spec(__fmul_rn(dtv, __ldg(p.A + h)));
    }

    LaneThreshold<FMT, RULE, LPR> thr;
    thr.init(p.weyl, step_t, lis);
    const uint32_t key0 = (uint32_t)p.sr_seed, key1 = (uint32_t)(p.sr_seed >> 32);

    const uint32_t hash_base = step_t * kHashP2 + p.layer * kHashP3 + key0 * kHashP4;
    const uint32_t p_first = sub * p.rps;                         // first row of this slot inside the item
    const uint64_t row_first = (uint64_t)item * p.P + p_first;    // local row index (this call's tensors)
    const uint64_t grow_first = row_first + p.row_off0 + (uint64_t)b * p.row_skip;   // global row index
    uint4* state = reinterpret_cast<uint4*>(p.state);
    const bool row_scale = Fmt<FMT>::kScaled && (p.scale_block == (uint32_t)N);

    float ykeep = 0.0f;
    for (uint32_t k0 = 0; k0 < p.rps; k0 += UNR) {
        uint4 raw[UNR];
        float xv[UNR];
        float sc[UNR];
        bool ok[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const uint32_t k = k0 + u;
            ok[u] = item_ok && (k < p.rps) && (p_first + k < p.P);
            if (ok[u]) {        // debug builds: the row's vector, x / y element and scale must lie inside the caller's buffers
                ok[u] = SSDQ_RANGE_OK(p, DBG_STATE, (row_first + k) * LPR + lis, 1, state_vecs) && SSDQ_RANGE_OK(p, DBG_ROWS, row_first + k, 1, rows);
                if constexpr (Fmt<FMT>::kScaled)
                    ok[u] = ok[u] && SSDQ_RANGE_OK(p, DBG_SCALES, row_scale ? row_first + k : (row_first + k) * (N / 16) + lis, 1, scales);
            }
            raw[u] = make_uint4(0u, 0u, 0u, 0u);
            xv[u] = 0.0f;
            sc[u] = 0.0f;
            if (ok[u]) {
                const uint64_t row = row_first + k;
                raw[u] = state[row * LPR + lis];
                xv[u] = __ldg(p.x + row);
                if constexpr (Fmt<FMT>::kScaled)
                    sc[u] = row_scale ? p.scales[row] : p.scales[row * (N / 16) + lis];
            }
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const uint32_t k = k0 + u;
            const uint64_t row = row_first + k;
            float hv[EPL];
            unpack_lane<FMT>(raw[u], hv);
            const float dtx = __fmul_rn(dtv, xv[u]);
            float dot = 0.0f;
            float amax = 0.0f;
#pragma unroll
            for (int j = 0; j < EPL; ++j) {
                float hin = hv[j];
                if constexpr (Fmt<FMT>::kScaled) hin = __fmul_rn(hin, sc[u]);
                const float w = __fmul_rn(dtx, Bv[j]);
                const float hn = __fmaf_rn(APS ? av[APS ? j : 0] : av[0], hin, w);
                hv[j] = hn;
                dot = __fmaf_rn(Cv[j], hn, dot);
                if constexpr (Fmt<FMT>::kScaled) amax = fmaxf(amax, fabsf(hn));
            }
            // readout: reduce the partial dots over the slot
#pragma unroll
            for (int off = LPR / 2; off > 0; off >>= 1) dot += __shfl_xor_sync(FULL, dot, off);
            if constexpr (Fmt<FMT>::kScaled) {
                if (row_scale) {
#pragma unroll
                    for (int off = LPR / 2; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, off));
                }
                const float s = fmaxf(__fdiv_rn(amax, p.scale_top), 1.17549435e-38f);
                const float rinv = __frcp_rn(s);
#pragma unroll
                for (int j = 0; j < EPL; ++j) hv[j] = __fmul_rn(hv[j], rinv);
                if (ok[u]) {
                    if (row_scale) { if (lis == 0) p.scales[row] = s; }
                    else p.scales[row * (N / 16) + lis] = s;
                }
            }
            uint32_t g_lo = 0, g_hi = 0, acc0 = 0;
            if constexpr (RULE == RULE_WEYL) acc0 = thr.weyl_acc0(grow_first + k);
            if constexpr (RULE == RULE_SR_HASH) acc0 = thr.hash_key0(grow_first + k, hash_base, key1);
            if constexpr (RULE == RULE_SR) thr.sr_group(grow_first + k, g_lo, g_hi);
            const uint4 packed = round_pack_lane<FMT, RULE>(hv, acc0, p.weyl.mul_col, g_lo, g_hi, step_t, p.layer,
                                                             key0, key1, p.scale_top);
            if (ok[u]) state[row * LPR + lis] = packed;
            // y: lane (k mod LPR) of the slot keeps row k; flushed every LPR rows
            const float yv = __fmaf_rn(Dv, xv[u], dot);
            if ((k % LPR) == lis) ykeep = yv;
            const bool last_of_batch = ((k % LPR) == LPR - 1) || (k + 1 == p.rps);
            if (last_of_batch) {
                const uint32_t kb = k - (k % LPR);                // first row of this batch of <= LPR rows
                const uint32_t kk = kb + lis;
                if (item_ok && kk <= k && kk < p.rps && (p_first + kk < p.P))
                    p.y[row_first + kk] = p.z ? __fmul_rn(ykeep, silu(__ldg(p.z + row_first + kk))) : ykeep;
            }
        }
    }
}

// Sum four per-lane partial dots over the LPR lanes of a slot with a transposed butterfly: after
// the first two exchanges each lane carries one of the four rows, so the remaining steps move one
// value instead of four.  Returns the total of row j = lane_in_slot / (LPR / 4).
template <int LPR>
__device__ __forceinline__ float reduce4_over_slot(float d0, float d1, float d2, float d3, uint32_t lis) {
    static_assert(LPR >= 4, "needs at least four lanes per row");
    constexpr unsigned FULL = 0xFFFFFFFFu;
    const bool hi1 = (lis & (LPR / 2)) != 0;
    float k0 = hi1 ? d2 : d0, k1 = hi1 ? d3 : d1;
    const float s0 = hi1 ? d0 : d2, s1 = hi1 ? d1 : d3;
    k0 += __shfl_xor_sync(FULL, s0, LPR / 2);
    k1 += __shfl_xor_sync(FULL, s1, LPR / 2);
    const bool hi2 = (lis & (LPR / 4)) != 0;
    float k = hi2 ? k1 : k0;
    const float s = hi2 ? k0 : k1;
    k += __shfl_xor_sync(FULL, s, LPR / 4);
#pragma unroll
    for (int off = LPR / 8; off > 0; off >>= 1) k += __shfl_xor_sync(FULL, k, off);
    return k;
}

// cp.async.wait_group needs an immediate: allow at most RPS - 1 - k groups (the rows after k) to be pending.
template <int RPS>
__device__ __forceinline__ void cp_async_wait_rows(int k) {
    static_assert(RPS <= 16, "one commit group per row, at most 16 rows per lane");
    switch (RPS - 1 - k) {
        case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
        case 7: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
        case 8: asm volatile("cp.async.wait_group 8;" ::: "memory"); break;
        case 9: asm volatile("cp.async.wait_group 9;" ::: "memory"); break;
        case 10: asm volatile("cp.async.wait_group 10;" ::: "memory"); break;
        case 11: asm volatile("cp.async.wait_group 11;" ::: "memory"); break;
        case 12: asm volatile("cp.async.wait_group 12;" ::: "memory"); break;
        case 13: asm volatile("cp.async.wait_group 13;" ::: "memory"); break;
        case 14: asm volatile("cp.async.wait_group 14;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 15;" ::: "memory"); break;
    }
}

// The same for two rows (slots of at least two lanes): returns the total of row j = lane_in_slot / (LPR / 2).
template <int LPR>
__device__ __forceinline__ float reduce2_over_slot(float d0, float d1, uint32_t lis) {
    static_assert(LPR >= 2, "needs at least two lanes per row");
    constexpr unsigned FULL = 0xFFFFFFFFu;
    const bool hi = (lis & (LPR / 2)) != 0;
    float k = hi ? d1 : d0;
    const float s = hi ? d0 : d1;
    k += __shfl_xor_sync(FULL, s, LPR / 2);
#pragma unroll
    for (int off = LPR / 4; off > 0; off >>= 1) k += __shfl_xor_sync(FULL, k, off);
    return k;
}

// The tile kernel: the same computation for the shapes that dominate (one decay per head, a head of
// P = (kThreads / LPR) * RPS rows), one CTA per (b, h).  A head's state is one contiguous tile (16 KB for
// 64 x 128 two-byte codes), staged through shared memory; rows are walked GRP = min(4, RPS) at a time so that their
// readout dots share one transposed reduction.  No guards, no idle lanes.
// EXTRAS: any of dt_bias, in-kernel softplus, B/C groups or the z gate is in use (the plain step pays nothing for them).
template <int FMT, int RULE, int LPR, int RPS, bool EXTRAS>
__global__ void __launch_bounds__(kThreads) ssd_update_tile_kernel(const UpdateParams p) {
    grid_dependency_gate(p.overlap);
    constexpr int EPL = Fmt<FMT>::kEpl;
    constexpr int N = LPR * EPL;
    constexpr int NSLOT = kThreads / LPR;
    constexpr unsigned FULL = 0xFFFFFFFFu;
    constexpr int GRP = RPS >= 4 ? 4 : 2;        // rows per reduction group
    static_assert(RPS % GRP == 0 && LPR >= GRP, "rows are processed GRP at a time by slots of at least GRP lanes");

    const uint32_t step_t = p.step_t + (p.step_base ? __ldcg(p.step_base) : 0u);
    const uint32_t lis = threadIdx.x % LPR;
    const uint32_t slot = threadIdx.x / LPR;
    const uint32_t h = blockIdx.x;                  // grid = (H, B): no index division
    const uint32_t b = blockIdx.y;
    const uint32_t item = b * p.H + h;
    const uint32_t n0 = lis * EPL;
    const uint64_t row_first = (uint64_t)item * (NSLOT * RPS) + slot * RPS;
    const bool row_scale = Fmt<FMT>::kScaled && (p.scale_block == (uint32_t)N);

    // every load of the CTA is issued here
    // The state tile goes global -> shared with asynchronous 16-byte copies, one commit group per row: the bytes in
    // flight cost no registers (more CTAs per SM, hence more of them), and row k can be consumed as soon as it has
    // landed while the later rows are still on their way.  Each lane reads back only what it copied itself, so
    // cp.async.wait_group is all the synchronisation needed.
    __shared__ uint4 tile[RPS][kThreads];
    uint4* sp = reinterpret_cast<uint4*>(p.state) + row_first * LPR + lis;
    // debug builds: everything this lane will touch, checked once (a lane that fails keeps running but accesses nothing)
    bool mem_ok = SSDQ_RANGE_OK(p, DBG_STATE, row_first * LPR + lis, (RPS - 1) * LPR + 1, state_vecs) &&
                  SSDQ_RANGE_OK(p, DBG_ROWS, row_first, RPS, rows) && SSDQ_RANGE_OK(p, DBG_ITEMS, item, 1, items) &&
                  SSDQ_RANGE_OK(p, DBG_BC, (size_t)b * ((EXTRAS && p.ngroups > 1) ? p.ngroups : 1u) * N + n0, EPL, bc_floats);
    if constexpr (Fmt<FMT>::kScaled)
        mem_ok = mem_ok && SSDQ_RANGE_OK(p, DBG_SCALES, row_scale ? row_first : row_first * (N / 16) + lis, row_scale ? RPS : (RPS - 1) * (N / 16) + 1, scales);
#pragma unroll
    for (int k = 0; k < RPS; ++k) {
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(&tile[k][threadIdx.x]);
        if (mem_ok) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n cp.async.commit_group;" ::"r"(dst), "l"(sp + k * LPR) : "memory");
    }
    float xv[RPS];
    float sc[Fmt<FMT>::kScaled ? RPS : 1];
#pragma unroll
    for (int k = 0; k < RPS / GRP; ++k) {
        if (!mem_ok) {
            xv[GRP * k] = 0.0f; xv[GRP * k + 1] = 0.0f;
            if constexpr (GRP == 4) { xv[4 * k + 2] = 0.0f; xv[4 * k + 3] = 0.0f; }
        } else if constexpr (GRP == 4) {
            const float4 x4 = __ldg(reinterpret_cast<const float4*>(p.x + row_first) + k);
            xv[4 * k] = x4.x; xv[4 * k + 1] = x4.y; xv[4 * k + 2] = x4.z; xv[4 * k + 3] = x4.w;
        } else {
            const float2 x2 = __ldg(reinterpret_cast<const float2*>(p.x + row_first) + k);
            xv[2 * k] = x2.x; xv[2 * k + 1] = x2.y;
        }
    }
    if constexpr (Fmt<FMT>::kScaled) {
#pragma unroll
        for (int k = 0; k < RPS; ++k) sc[k] = !mem_ok ? 0.0f : row_scale ? p.scales[row_first + k] : p.scales[(row_first + k) * (N / 16) + lis];
    }
    f32x2 B2[EPL / 2], C2[EPL / 2];
    {
        const size_t grp = (!EXTRAS || p.ngroups == 1) ? (size_t)b : (size_t)b * p.ngroups + h / p.heads_per_group;
        const float4* Bp = reinterpret_cast<const float4*>(p.Bm + grp * N + n0);
        const float4* Cp = reinterpret_cast<const float4*>(p.Cm + grp * N + n0);
#pragma unroll
        for (int i = 0; i < EPL / 4; ++i) {
            const float4 zero4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            const float4 bb = mem_ok ? __ldg(Bp + i) : zero4, cc = mem_ok ? __ldg(Cp + i) : zero4;
            B2[2 * i] = pack2(bb.x, bb.y); B2[2 * i + 1] = pack2(bb.z, bb.w);
            C2[2 * i] = pack2(cc.x, cc.y); C2[2 * i + 1] = pack2(cc.z, cc.w);
        }
    }
    float dtv = mem_ok ? __ldg(p.dt + item) : 0.0f;
    if constexpr (EXTRAS) {
        if (p.dt_bias) dtv = __fadd_rn(dtv, __ldg(p.dt_bias + h));
        if (p.dt_softplus) dtv = softplus_spec(dtv);
    }
    // the lanes that will write y fetch their gate values now (row j = lane_in_slot / (LPR / GRP) of each group)
    const bool y_writer = (lis & (LPR / GRP - 1)) == 0;
    float gate[RPS / GRP];
#pragma unroll
    for (int g4 = 0; g4 < RPS / GRP; ++g4)
        gate[g4] = (EXTRAS && p.z && y_writer && mem_ok) ? __ldg(p.z + row_first + g4 * GRP + lis / (LPR / GRP)) : 0.0f;
    const float a = exp_spec(__fmul_rn(dtv, __ldg(p.A + h)));
    const f32x2 a2 = pack2(a, a);
    const float Dl = (p.D && lis == 0) ? __ldg(p.D + h) : 0.0f;     // the skip term enters the dot on one lane

    LaneThreshold<FMT, RULE, LPR> thr;
    thr.init(p.weyl, step_t, lis);
    const uint32_t key0 = (uint32_t)p.sr_seed, key1 = (uint32_t)(p.sr_seed >> 32);
    const uint64_t grow_first = row_first + p.row_off0 + (uint64_t)b * p.row_skip;
    uint32_t acc_row = 0;
    uint64_t grp_row = 0;
    const uint32_t hash_base = step_t * kHashP2 + p.layer * kHashP3 + key0 * kHashP4;
    if constexpr (RULE == RULE_WEYL) acc_row = thr.weyl_acc0(grow_first);
    if constexpr (RULE == RULE_SR) grp_row = (grow_first * (uint64_t)N + n0) >> 2;

#pragma unroll
    for (int g4 = 0; g4 < RPS / GRP; ++g4) {
        float dots[GRP];
#pragma unroll
        for (int u = 0; u < GRP; ++u) {
            const int k = g4 * GRP + u;
            float hv[EPL];
            cp_async_wait_rows<RPS>(k);                       // rows 0..k have landed
            unpack_lane<FMT>(tile[k][threadIdx.x], hv);
            // Eq. 1 and the partial readout, two entries per instruction (packed binary32: the same operations and roundings)
            const float dtx = __fmul_rn(dtv, xv[k]);
            const f32x2 dtx2 = pack2(dtx, dtx);
            f32x2 dot2 = pack2(__fmul_rn(Dl, xv[k]), 0.0f);
            float amax = 0.0f;
            f32x2 hn2[EPL / 2];
#pragma unroll
            for (int i = 0; i < EPL / 2; ++i) {
                f32x2 hin = pack2(hv[2 * i], hv[2 * i + 1]);
                if constexpr (Fmt<FMT>::kScaled) hin = mul2_rn(hin, pack2(sc[k], sc[k]));
                const f32x2 hn = fma2_rn(a2, hin, mul2_rn(dtx2, B2[i]));
                hn2[i] = hn;
                dot2 = fma2_rn(C2[i], hn, dot2);
                unpack2(hn, hv[2 * i], hv[2 * i + 1]);
                if constexpr (Fmt<FMT>::kScaled) amax = max3abs(amax, hv[2 * i], hv[2 * i + 1]);
            }
            {
                float d0, d1;
                unpack2(dot2, d0, d1);
                dots[u] = __fadd_rn(d0, d1);
            }
            if constexpr (Fmt<FMT>::kScaled) {
                if (row_scale) {
#pragma unroll
                    for (int off = LPR / 2; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, off));
                }
                const float s = fmaxf(__fdiv_rn(amax, p.scale_top), 1.17549435e-38f);
                const float rinv = __frcp_rn(s);
                const f32x2 rinv2 = pack2(rinv, rinv);
#pragma unroll
                for (int i = 0; i < EPL / 2; ++i) unpack2(mul2_rn(hn2[i], rinv2), hv[2 * i], hv[2 * i + 1]);
                if (row_scale) { if (lis == 0 && mem_ok) p.scales[row_first + k] = s; }
                else if (mem_ok) p.scales[(row_first + k) * (N / 16) + lis] = s;
            }
            if constexpr (RULE == RULE_SR_HASH) acc_row = thr.hash_key0(grow_first + k, hash_base, key1);
            const uint4 packed = round_pack_lane<FMT, RULE>(hv, acc_row, p.weyl.mul_col, (uint32_t)grp_row,
                                                             (uint32_t)(grp_row >> 32), step_t, p.layer, key0, key1, p.scale_top);
            if (mem_ok) sp[k * LPR] = packed;
            if constexpr (RULE == RULE_WEYL) acc_row += thr.row_mul;
            if constexpr (RULE == RULE_SR) grp_row += N / 4;
        }
        float tot;
        if constexpr (GRP == 4) tot = reduce4_over_slot<LPR>(dots[0], dots[1], dots[2], dots[3], lis);
        else tot = reduce2_over_slot<LPR>(dots[0], dots[1], lis);
        if (y_writer && mem_ok) p.y[row_first + g4 * GRP + lis / (LPR / GRP)] = (EXTRAS && p.z) ? __fmul_rn(tot, silu(gate[g4])) : tot;
    }
}

// The persistent kernel of ssdq_stream.cuh, for the shapes it covers; `launched` says whether it took the call.
template <int FMT, int RULE, int LPR>
cudaError_t try_launch_stream(const UpdateParams& p, cudaStream_t stream, bool& launched);

// The kernel of ssdq_mamba1.cuh (N = 16, headdim 1, one decay per state), for the calls it covers.
template <int FMT, int RULE>
cudaError_t try_launch_mamba1(const UpdateParams& p, cudaStream_t stream, bool& launched);

// The kernel of ssdq_headscale.cuh (one scale per (sequence, head)), for the shapes it covers.
template <int FMT, int RULE, int LPR>
cudaError_t try_launch_headscale(const UpdateParams& p, cudaStream_t stream, bool& launched);

// Host-side launcher for one (format, rule): picks the lanes-per-row instantiation from N.
template <int FMT, int RULE, int LPR, bool APS>
inline cudaError_t launch_update_one(const UpdateParams& p, cudaStream_t stream) {
    UpdateParams q = p;
    const uint32_t nslot = kThreads / LPR;
    if constexpr (APS && FMT != FMT_FP32 && LPR * Fmt<FMT>::kEpl == 16) {
        bool launched = false;
        const cudaError_t e = try_launch_mamba1<FMT, RULE>(q, stream, launched);
        if (launched || e != cudaSuccess) return e;
    }
    if constexpr (Fmt<FMT>::kScaled) {
        if (q.scale_block == q.P * q.N && q.scale_block != q.N) {       // one scale per head: its own kernel or nothing
            bool launched = false;
            cudaError_t e = cudaErrorInvalidValue;
            if constexpr (!APS && LPR >= 4 && Fmt<FMT>::kBytes == 1) e = try_launch_headscale<FMT, RULE, LPR>(q, stream, launched);
            return launched ? e : cudaErrorInvalidValue;
        }
    }
    if constexpr (!APS && LPR >= 4 && Fmt<FMT>::kScaled && Fmt<FMT>::kBytes == 1) {
        bool launched = false;
        const cudaError_t e = try_launch_stream<FMT, RULE, LPR>(q, stream, launched);
        if (launched || e != cudaSuccess) return e;
    }
    if constexpr (!APS && LPR >= 4 && FMT != FMT_FP32) {
        // shapes the tile kernel covers: a head of nslot * {2, 4, 8, 16} rows; x, y (and row scales) 16-byte aligned
        const bool aligned = ((reinterpret_cast<uintptr_t>(q.x) | reinterpret_cast<uintptr_t>(q.y)) & 15u) == 0 &&
                             (!Fmt<FMT>::kScaled || (reinterpret_cast<uintptr_t>(q.scales) & 15u) == 0);
        const dim3 tile_grid(q.H, q.B);
        const bool extras = q.dt_bias || q.dt_softplus || q.z || q.ngroups > 1;
        if (aligned && q.B <= 65535u) {
#define SSDQ_TILE_CASE(R)                                                                                          \
            if (q.P == nslot * (R)) {                                                                              \
                note_kernel(1);                                                                                    \
                if (q.prepare_only) return cudaSuccess;                                                            \
                if (extras) return launch_update_kernel(ssd_update_tile_kernel<FMT, RULE, LPR, R, true>, tile_grid, 0, stream, q);  \
                return launch_update_kernel(ssd_update_tile_kernel<FMT, RULE, LPR, R, false>, tile_grid, 0, stream, q);             \
            }
            SSDQ_TILE_CASE(8u)
            SSDQ_TILE_CASE(4u)
            if constexpr (Fmt<FMT>::kBytes == 2) { SSDQ_TILE_CASE(16u) }     // P = 128 or N = 256 with two-byte codes
            if constexpr (Fmt<FMT>::kBytes == 1) { SSDQ_TILE_CASE(2u) }      // small heads with one-byte codes
#undef SSDQ_TILE_CASE
        }
    }
    uint32_t spi = 1;
    while (spi < q.P && spi < nslot) spi <<= 1;        // slots per item: power of two, >= min(P, nslot)
    q.spi = spi;
    q.items_per_cta = nslot / spi;
    q.rps = (q.P + spi - 1) / spi;
    const uint32_t grid = (q.n_items + q.items_per_cta - 1) / q.items_per_cta;
    note_kernel(0);
    if (q.prepare_only) return cudaSuccess;
    return launch_update_kernel(ssd_update_kernel<FMT, RULE, LPR, APS>, dim3(grid), 0, stream, q);
}

template <int FMT, int RULE, bool APS>
inline cudaError_t launch_update_n(const UpdateParams& p, cudaStream_t stream) {
    constexpr int EPL = Fmt<FMT>::kEpl;
    if (p.N % EPL != 0) return cudaErrorInvalidValue;
    switch (p.N / EPL) {   // lanes per row; N = LPR * EPL must be one of 16, 32, 64, 128, 256 and LPR <= 32
        case 1: if constexpr (EPL == 16) return launch_update_one<FMT, RULE, 1, APS>(p, stream); break;
        case 2: if constexpr (EPL >= 8) return launch_update_one<FMT, RULE, 2, APS>(p, stream); break;
        case 4: return launch_update_one<FMT, RULE, 4, APS>(p, stream);
        case 8: return launch_update_one<FMT, RULE, 8, APS>(p, stream);
        case 16: return launch_update_one<FMT, RULE, 16, APS>(p, stream);
        case 32: if constexpr (EPL <= 8) return launch_update_one<FMT, RULE, 32, APS>(p, stream); break;
        default: break;
    }
    return cudaErrorInvalidValue;
}

template <int FMT>
inline cudaError_t launch_update_fmt(const UpdateParams& p, int rule, bool aps, cudaStream_t stream) {
    if constexpr (FMT == FMT_FP32) {
        return aps ? launch_update_n<FMT, RULE_RTN, true>(p, stream) : launch_update_n<FMT, RULE_RTN, false>(p, stream);
    } else {
        switch (rule) {
            case RULE_RTN: return aps ? launch_update_n<FMT, RULE_RTN, true>(p, stream) : launch_update_n<FMT, RULE_RTN, false>(p, stream);
            case RULE_SR: return aps ? launch_update_n<FMT, RULE_SR, true>(p, stream) : launch_update_n<FMT, RULE_SR, false>(p, stream);
            case RULE_WEYL: return aps ? launch_update_n<FMT, RULE_WEYL, true>(p, stream) : launch_update_n<FMT, RULE_WEYL, false>(p, stream);
            case RULE_SR_HASH: return aps ? launch_update_n<FMT, RULE_SR_HASH, true>(p, stream) : launch_update_n<FMT, RULE_SR_HASH, false>(p, stream);
            default: return cudaErrorInvalidValue;
        }
    }
}

}  // namespace ssdq

// ssdq_headscale.cuh -- the fused decode step for one-byte stores that keep ONE FP32 scale per (sequence, head)
// instead of one per row or per 16 entries (scale_block = P * N).
//
// The scale of a write is max|h'| over the whole head / top, so nothing can be rounded before every row of the head
// has been updated: one CTA owns one (b, h), each lane keeps the updated values of its RPS rows (RPS x 16 binary32) in
// registers, the CTA reduces the maximum through shared memory, and only then are the rows scaled, rounded (Eq. 2) and
// stored.  Everything else -- thread mapping, asynchronous tile copy, operation order, thresholds -- is that of
// ssd_update_tile_kernel.
#pragma once
#include "ssdq_update.cuh"

namespace ssdq {

template <int FMT, int RULE, int LPR, int RPS>
__global__ void __launch_bounds__(kThreads) ssd_update_headscale_kernel(const UpdateParams p) {
    grid_dependency_gate(p.overlap);
    static_assert(Fmt<FMT>::kScaled && Fmt<FMT>::kEpl == 16, "one-byte block-scaled stores");
    constexpr int EPL = 16;
    constexpr int N = LPR * EPL;
    constexpr int NSLOT = kThreads / LPR;
    constexpr unsigned FULL = 0xFFFFFFFFu;
    constexpr int GRP = RPS >= 4 ? 4 : 2;
    static_assert(RPS % GRP == 0 && LPR >= GRP && RPS <= 8, "rows are reduced GRP at a time; at most 8 rows per lane stay in registers");

    const uint32_t step_t = p.step_t + (p.step_base ? __ldcg(p.step_base) : 0u);
    const uint32_t lis = threadIdx.x % LPR;
    const uint32_t slot = threadIdx.x / LPR;
    const uint32_t h = blockIdx.x, b = blockIdx.y;
    const uint32_t item = b * p.H + h;
    const uint32_t n0 = lis * EPL;
    const uint64_t row_first = (uint64_t)item * (NSLOT * RPS) + slot * RPS;

    __shared__ uint4 tile[RPS][kThreads];
    __shared__ float warp_max[kThreads / 32];
    uint4* sp = reinterpret_cast<uint4*>(p.state) + row_first * LPR + lis;
    // debug builds: everything this lane will touch, checked once (a lane that fails keeps running but accesses nothing)
    const bool mem_ok = SSDQ_RANGE_OK(p, DBG_STATE, row_first * LPR + lis, (RPS - 1) * LPR + 1, state_vecs) &&
                        SSDQ_RANGE_OK(p, DBG_ROWS, row_first, RPS, rows) && SSDQ_RANGE_OK(p, DBG_ITEMS, item, 1, items) &&
                        SSDQ_RANGE_OK(p, DBG_SCALES, item, 1, scales) && SSDQ_RANGE_OK(p, DBG_BC, (size_t)b * N + n0, EPL, bc_floats);
#pragma unroll
    for (int k = 0; k < RPS; ++k) {
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(&tile[k][threadIdx.x]);
        if (mem_ok) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n cp.async.commit_group;" ::"r"(dst), "l"(sp + k * LPR) : "memory");
    }
    float xv[RPS];
#pragma unroll
    for (int k = 0; k < RPS / 2; ++k) {
        const float2 x2 = mem_ok ? __ldg(reinterpret_cast<const float2*>(p.x + row_first) + k) : make_float2(0.0f, 0.0f);
        xv[2 * k] = x2.x; xv[2 * k + 1] = x2.y;
    }
    const float sc_old = mem_ok ? p.scales[item] : 0.0f;
    f32x2 B2[EPL / 2], C2[EPL / 2];
    {
        const float4* Bp = reinterpret_cast<const float4*>(p.Bm + (size_t)b * N + n0);
        const float4* Cp = reinterpret_cast<const float4*>(p.Cm + (size_t)b * N + n0);
#pragma unroll
        for (int i = 0; i < EPL / 4; ++i) {
            const float4 zero4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            const float4 bb = mem_ok ? __ldg(Bp + i) : zero4, cc = mem_ok ? __ldg(Cp + i) : zero4;
            B2[2 * i] = pack2(bb.x, bb.y); B2[2 * i + 1] = pack2(bb.z, bb.w);
            C2[2 * i] = pack2(cc.x, cc.y); C2[2 * i + 1] = pack2(cc.z, cc.w);
        }
    }
    const float dtv = mem_ok ? __ldg(p.dt + item) : 0.0f;
    const float a = exp_spec(__fmul_rn(dtv, __ldg(p.A + h)));
    const float Dl = (p.D && lis == 0) ? __ldg(p.D + h) : 0.0f;
    const f32x2 a2 = pack2(a, a), sc2 = pack2(sc_old, sc_old);
    const bool y_writer = (lis & (LPR / GRP - 1)) == 0;

    // pass 1: Eq. 1 and the readout for every row of the head; the updated values stay in registers
    f32x2 hn[RPS][EPL / 2];
    float amax = 0.0f;
#pragma unroll
    for (int g = 0; g < RPS / GRP; ++g) {
        float dots[GRP];
#pragma unroll
        for (int u = 0; u < GRP; ++u) {
            const int k = g * GRP + u;
            cp_async_wait_rows<RPS>(k);
            const uint4 raw = tile[k][threadIdx.x];
            const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float f[4];
                if constexpr (FMT == FMT_E4M3) unpack4_e4m3(rw[i], f);
                else unpack4_int8(rw[i], f);
                hn[k][2 * i] = pack2(f[0], f[1]);
                hn[k][2 * i + 1] = pack2(f[2], f[3]);
            }
            const float dtx = __fmul_rn(dtv, xv[k]);
            const f32x2 dtx2 = pack2(dtx, dtx);
            f32x2 dot2 = pack2(__fmul_rn(Dl, xv[k]), 0.0f);
#pragma unroll
            for (int i = 0; i < EPL / 2; ++i) {
                const f32x2 v = fma2_rn(a2, mul2_rn(hn[k][i], sc2), mul2_rn(dtx2, B2[i]));
                hn[k][i] = v;
                dot2 = fma2_rn(C2[i], v, dot2);
                float e0, e1;
                unpack2(v, e0, e1);
                amax = max3abs(amax, e0, e1);
            }
            float d0, d1;
            unpack2(dot2, d0, d1);
            dots[u] = __fadd_rn(d0, d1);
        }
        float tot;
        if constexpr (GRP == 4) tot = reduce4_over_slot<LPR>(dots[0], dots[1], dots[2], dots[3], lis);
        else tot = reduce2_over_slot<LPR>(dots[0], dots[1], lis);
        if (y_writer && mem_ok) p.y[row_first + g * GRP + lis / (LPR / GRP)] = tot;
    }
    // the head's maximum: warp shuffle, then across the warps through shared memory
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, off));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x / 32] = amax;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) amax = fmaxf(amax, warp_max[w]);
    const float s = fmaxf(__fdiv_rn(amax, p.scale_top), 1.17549435e-38f);
    const float rinv = __frcp_rn(s);
    const f32x2 rinv2 = pack2(rinv, rinv);
    if (threadIdx.x == 0 && mem_ok) p.scales[item] = s;

    // pass 2: scale, thresholds, Eq. 2, store
    LaneThreshold<FMT, RULE, LPR> thr;
    thr.init(p.weyl, step_t, lis);
    const uint32_t key0 = (uint32_t)p.sr_seed, key1 = (uint32_t)(p.sr_seed >> 32);
    const uint32_t hash_base = step_t * kHashP2 + p.layer * kHashP3 + key0 * kHashP4;
    const uint64_t grow_first = row_first + p.row_off0 + (uint64_t)b * p.row_skip;
    uint32_t acc_row = 0;
    uint64_t grp_row = 0;
    if constexpr (RULE == RULE_WEYL) acc_row = thr.weyl_acc0(grow_first);
    if constexpr (RULE == RULE_SR) grp_row = (grow_first * (uint64_t)N + n0) >> 2;
#pragma unroll
    for (int k = 0; k < RPS; ++k) {
        float v[EPL];
#pragma unroll
        for (int i = 0; i < EPL / 2; ++i) unpack2(mul2_rn(hn[k][i], rinv2), v[2 * i], v[2 * i + 1]);
        if constexpr (RULE == RULE_SR_HASH) acc_row = thr.hash_key0(grow_first + k, hash_base, key1);
        const uint4 packed = round_pack_lane<FMT, RULE>(v, acc_row, p.weyl.mul_col, (uint32_t)grp_row, (uint32_t)(grp_row >> 32), step_t,
                                                 p.layer, key0, key1, p.scale_top);
        if (mem_ok) sp[k * LPR] = packed;
        if constexpr (RULE == RULE_WEYL) acc_row += thr.row_mul;
        if constexpr (RULE == RULE_SR) grp_row += N / 4;
    }
}

// Shapes covered: heads of (kThreads / LPR) * {2, 4, 8} rows, the plain signature, x and y 8-byte aligned.
template <int FMT, int RULE, int LPR>
cudaError_t try_launch_headscale(const UpdateParams& p, cudaStream_t stream, bool& launched) {
    launched = false;
    if constexpr (LPR >= 4 && Fmt<FMT>::kScaled && Fmt<FMT>::kBytes == 1) {
        const bool extras = p.dt_bias || p.dt_softplus || p.z || p.ngroups > 1;
        const bool aligned = ((reinterpret_cast<uintptr_t>(p.x) | reinterpret_cast<uintptr_t>(p.y)) & 7u) == 0;
        constexpr uint32_t nslot = kThreads / LPR;
        if (extras || !aligned || p.B > 65535u) return cudaSuccess;
        const dim3 grid(p.H, p.B);
#define SSDQ_HEAD_CASE(R)                                                                          \
        if (p.P == nslot * (R)) {                                                                  \
            launched = true;                                                                       \
            note_kernel(3);                                                                        \
            if (p.prepare_only) return cudaSuccess;                                                \
            return launch_update_kernel(ssd_update_headscale_kernel<FMT, RULE, LPR, R>, grid, 0, stream, p); \
        }
        SSDQ_HEAD_CASE(4u)
        SSDQ_HEAD_CASE(8u)
        SSDQ_HEAD_CASE(2u)
#undef SSDQ_HEAD_CASE
    }
    return cudaSuccess;
}

}  // namespace ssdq

// ssdq_mamba1.cuh -- the fused decode step for the Mamba-1 state layout: [B, d_inner, N = 16] per layer (headdim 1),
// one decay PER STATE, a = exp(dt * A[d, n]) (Appendix B "Runners": the Mamba-1 selective scan evaluated step by step).
//
// Here every entry needs its own exponential, so the step is bound by arithmetic as much as by memory, and rows are
// only 16 entries long.  One lane owns one whole row (b, d): no shuffle is needed for the readout or the block maximum,
// the channel's 16 values of A stay in registers while the CTA walks over the batch, and the exponential and Eq. 1 are
// issued two entries at a time with the packed binary32 instructions.  Consecutive lanes own consecutive channels, so
// the state, dt, x and y accesses of a warp are contiguous.
#pragma once
#include <cstddef>
#include <type_traits>
#include "ssdq_update.cuh"

namespace ssdq {

// exp_spec on two values at once: the same operations in the same order as exp_spec, bit for bit.  rint is taken by
// adding and subtracting 1.5 * 2^23 with SCALAR adds (a packed add after the packed multiply would be contracted into a
// fused multiply-add by the assembler and could move k); the integer k then sits in the low bits of the sum.
__device__ __forceinline__ f32x2 exp_spec2(f32x2 z2) {
    {
        float z0, z1;
        unpack2(z2, z0, z1);
        z2 = pack2(fminf(fmaxf(z0, -87.0f), 88.0f), fminf(fmaxf(z1, -87.0f), 88.0f));
    }
    float t0, t1;
    unpack2(mul2_rn(z2, pack2(0x1.715476p+0f, 0x1.715476p+0f)), t0, t1);
    const float m0 = __fadd_rn(t0, 12582912.0f), m1 = __fadd_rn(t1, 12582912.0f);       // nearest-even integer, |t| < 2^22
    const f32x2 k2 = add2_rn(pack2(m0, m1), pack2(-12582912.0f, -12582912.0f));         // exact; its inputs are sums, not products
    f32x2 r = fma2_rn(k2, pack2(-0x1.62e400p-1f, -0x1.62e400p-1f), z2);
    r = fma2_rn(k2, pack2(-0x1.7f7d1cp-20f, -0x1.7f7d1cp-20f), r);
    f32x2 p = pack2(0x1.a01a02p-13f, 0x1.a01a02p-13f);
    p = fma2_rn(p, r, pack2(0x1.6c16c2p-10f, 0x1.6c16c2p-10f));
    p = fma2_rn(p, r, pack2(0x1.111112p-7f, 0x1.111112p-7f));
    p = fma2_rn(p, r, pack2(0x1.555556p-5f, 0x1.555556p-5f));
    p = fma2_rn(p, r, pack2(0x1.555556p-3f, 0x1.555556p-3f));
    p = fma2_rn(p, r, pack2(0.5f, 0.5f));
    p = fma2_rn(p, r, pack2(1.0f, 1.0f));
    p = fma2_rn(p, r, pack2(1.0f, 1.0f));
    uint32_t p0, p1;
    unpack2u(p, p0, p1);
    return pack2u(p0 + (__float_as_uint(m0) << 23), p1 + (__float_as_uint(m1) << 23));    // exponent field += k
}

// grid = (ceil(H / kThreads), batch chunks); CTA (cx, cy) owns channels cx * kThreads .. and sequences
// [cy * b_per_cta, (cy + 1) * b_per_cta).  N = 16, P = 1, A is [H, 16].
//
// A lane works on one row at a time and a row is a long dependent computation, so the bytes of the NEXT row (its codes,
// dt, x, scale, and the sequence's B and C) are requested with asynchronous copies into a two-stage shared-memory ring
// before the current row is computed: the loads cost no registers and their latency hides behind the arithmetic.
// Each lane copies its own row; B and C of a sequence (128 bytes, the same for the whole warp) are copied once per warp
// by its first eight lanes.  Channels beyond H (last tile only) run on a clamped channel and store nothing.
// With the loads out of the way the kernel is bound by instruction issue (every entry needs its own exponential), so
// the dithered rules, which need more registers, trade two resident CTAs for a spill-free loop (measured).
// The loop is unrolled over the two stages so that every shared-memory address is a per-thread base plus a constant,
// and rows are addressed by a 32-bit index (B * H < 2^32) widened once per access: the ring costs ~25 instructions per row.
template <int SOFF, int GOFF>
__device__ __forceinline__ void cp_async16_ca_at(uint32_t smem_base, const void* gmem_base) {
    asm volatile("cp.async.ca.shared.global [%0 + %2], [%1 + %3], 16;" ::"r"(smem_base), "l"(gmem_base), "n"(SOFF), "n"(GOFF) : "memory");
}
template <int SOFF>
__device__ __forceinline__ void cp_async4_ca_at(uint32_t smem_base, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0 + %2], [%1], 4;" ::"r"(smem_base), "l"(gmem), "n"(SOFF) : "memory");
}

template <int CH>
struct Mamba1Stage {
    uint4 codes[CH][kThreads];
    float bc[kThreads / 32][32];        // per warp: B[0..15], C[0..15] of the sequence
    float dt[kThreads], x[kThreads], sc[kThreads];
};

template <int FMT, int RULE>
__global__ void __launch_bounds__(kThreads, RULE == RULE_RTN ? 8 : 6) ssd_update_mamba1_kernel(const UpdateParams p) {
    grid_dependency_gate(p.overlap);
    constexpr int EPL = Fmt<FMT>::kEpl;                 // entries per 16-byte chunk: 8 (two-byte codes) or 16
    constexpr int N = 16;
    constexpr int CH = N / EPL;                         // chunks per row: 2 or 1
    constexpr unsigned FULL = 0xFFFFFFFFu;
    using Stage = Mamba1Stage<CH>;
    __shared__ __align__(16) Stage ring[2];

    const uint32_t step_t = p.step_t + (p.step_base ? __ldcg(p.step_base) : 0u);
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t d_raw = blockIdx.x * kThreads + tid;
    const bool active = d_raw < p.H;
    const uint32_t d = active ? d_raw : p.H - 1u;
    const uint32_t b_first = blockIdx.y * p.rps;        // rps: sequences per CTA
    const uint32_t b_last = min(b_first + p.rps, p.B);
    if (b_first >= b_last) return;                      // the whole CTA

    f32x2 A2[N / 2];
    {
        const float4* Ap = reinterpret_cast<const float4*>(p.A + (size_t)d * N);
#pragma unroll
        for (int i = 0; i < N / 4; ++i) {
            const float4 a = __ldg(Ap + i);
            A2[2 * i] = pack2(a.x, a.y);
            A2[2 * i + 1] = pack2(a.z, a.w);
        }
    }
    const float Dv = p.D ? __ldg(p.D + d) : 0.0f;
    const uint32_t key0 = (uint32_t)p.sr_seed, key1 = (uint32_t)(p.sr_seed >> 32);
    const uint32_t hash_base = step_t * kHashP2 + p.layer * kHashP3 + key0 * kHashP4;
    // Weyl: a row is one dither block (block 16 = N): r = global row, c = n
    const uint32_t weyl_const = p.weyl.mul_row + p.weyl.mul_col + p.weyl.base + step_t * p.weyl.phi;

    const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(&ring[0]);
    const uint32_t t16 = ring_s + tid * 16u, t4 = ring_s + tid * 4u;                 // this thread's 16-byte and 4-byte cells
    const uint32_t bcw = ring_s + warp * 128u + (lane & 7u) * 16u;                   // lanes 0-7: one 16-byte chunk of the warp's B | C
    const float* bc_src = (lane < 4u ? p.Bm : p.Cm) + (lane & 3u) * 4u;
    const char* state_c = reinterpret_cast<const char*>(p.state);
    char* state_w = reinterpret_cast<char*>(p.state);
#ifdef SSDQ_DEBUG
    uint32_t ok_bits = 0;                               // bit s: the row in stage s passed the range checks
#endif

    auto issue = [&](uint32_t b, auto stage_c) {
        constexpr int S = decltype(stage_c)::value;
        constexpr int SO = S * (int)sizeof(Stage);
        const uint32_t row = b * p.H + d;
#ifdef SSDQ_DEBUG
        // the row's vectors, its x / y / dt elements, its scale and the sequence's B and C
        bool ok = SSDQ_RANGE_OK(p, DBG_STATE, (uint64_t)row * CH, CH, state_vecs) && SSDQ_RANGE_OK(p, DBG_ROWS, row, 1, rows) &&
                  SSDQ_RANGE_OK(p, DBG_ITEMS, row, 1, items) && SSDQ_RANGE_OK(p, DBG_BC, (size_t)b * N, N, bc_floats);
        if constexpr (Fmt<FMT>::kScaled) ok = ok && SSDQ_RANGE_OK(p, DBG_SCALES, row, 1, scales);
        ok = __all_sync(FULL, ok);                      // lanes meet at warp barriers and share B / C: skip as a warp
        ok_bits = (ok_bits & ~(1u << S)) | ((uint32_t)ok << S);
        if (!ok) return;
#endif
        // .ca: a two-byte row is two 16-byte chunks 32 bytes apart per lane, so each copy instruction touches every
        // sector of the warp's kilobyte; keeping the lines in L1 lets the second one hit there
        const char* sp = state_c + (uint64_t)row * (CH * 16u);
        cp_async16_ca_at<SO + (int)offsetof(Stage, codes), 0>(t16, sp);
        if constexpr (CH == 2) cp_async16_ca_at<SO + (int)offsetof(Stage, codes) + kThreads * 16, 16>(t16, sp);
        cp_async4_ca_at<SO + (int)offsetof(Stage, dt)>(t4, p.dt + row);
        cp_async4_ca_at<SO + (int)offsetof(Stage, x)>(t4, p.x + row);
        if constexpr (Fmt<FMT>::kScaled) cp_async4_ca_at<SO + (int)offsetof(Stage, sc)>(t4, p.scales + row);
        if (lane < 8u) cp_async16_ca_at<SO + (int)offsetof(Stage, bc), 0>(bcw, bc_src + (size_t)b * N);
    };

    auto row_step = [&](uint32_t b, auto stage_c) {
        constexpr int S = decltype(stage_c)::value;
        __syncwarp(FULL);                               // every lane is done with the B / C of the stage refilled next
        if (b + 1 < b_last) issue(b + 1, std::integral_constant<int, 1 - S>{});
        cp_async_commit();
        cp_async_wait<1>();                             // this row's group has landed (the next one may be pending)
        __syncwarp(FULL);                               // ... also the B / C chunks that other lanes copied
#ifdef SSDQ_DEBUG
        if (!((ok_bits >> S) & 1u)) return;             // the whole warp
#endif
        const Stage& st = ring[S];
        const uint32_t row = b * p.H + d;
        uint4 raw[CH];
#pragma unroll
        for (int c = 0; c < CH; ++c) raw[c] = st.codes[c][tid];
        const float dtv = st.dt[tid], xv = st.x[tid];
        float sc_old = 0.0f;
        if constexpr (Fmt<FMT>::kScaled) sc_old = st.sc[tid];
        const float4* Bp = reinterpret_cast<const float4*>(&st.bc[warp][0]);            // the same address in every lane: a broadcast
        const float4* Cp = Bp + N / 4;
        const float dtx = __fmul_rn(dtv, xv);
        const f32x2 dt2 = pack2(dtv, dtv), dtx2 = pack2(dtx, dtx), sc2 = pack2(sc_old, sc_old);
        float hin[N];
#pragma unroll
        for (int c = 0; c < CH; ++c) unpack_lane<FMT>(raw[c], hin + c * EPL);
        f32x2 hn[N / 2];
        f32x2 dot2 = pack2(__fmul_rn(Dv, xv), 0.0f);
        [[maybe_unused]] float amax = 0.0f;
#pragma unroll
        for (int i = 0; i < N / 4; ++i) {
            const float4 bb = Bp[i], cc = Cp[i];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int q = 2 * i + j;
                const f32x2 a2 = exp_spec2(mul2_rn(dt2, A2[q]));
                f32x2 h2 = pack2(hin[2 * q], hin[2 * q + 1]);
                if constexpr (Fmt<FMT>::kScaled) h2 = mul2_rn(h2, sc2);
                const f32x2 B2 = j ? pack2(bb.z, bb.w) : pack2(bb.x, bb.y);
                const f32x2 C2 = j ? pack2(cc.z, cc.w) : pack2(cc.x, cc.y);
                const f32x2 v = fma2_rn(a2, h2, mul2_rn(dtx2, B2));
                hn[q] = v;
                dot2 = fma2_rn(C2, v, dot2);
                if constexpr (Fmt<FMT>::kScaled) {
                    float e0, e1;
                    unpack2(v, e0, e1);
                    amax = max3abs(amax, e0, e1);
                }
            }
        }
        if (active) {
            float d0, d1;
            unpack2(dot2, d0, d1);
            p.y[row] = __fadd_rn(d0, d1);
        }
        float v[N];
        if constexpr (Fmt<FMT>::kScaled) {
            const float s = fmaxf(__fdiv_rn(amax, p.scale_top), 1.17549435e-38f);
            const float rinv = rcp_scale(s);
            const f32x2 rinv2 = pack2(rinv, rinv);
#pragma unroll
            for (int q = 0; q < N / 2; ++q) unpack2(mul2_rn(hn[q], rinv2), v[2 * q], v[2 * q + 1]);
            if (active) p.scales[row] = s;
        } else {
#pragma unroll
            for (int q = 0; q < N / 2; ++q) unpack2(hn[q], v[2 * q], v[2 * q + 1]);
        }
        // global row = local row + row_off0 + b * row_skip; the Weyl accumulator needs it modulo 2^32 only
        uint64_t flat0 = 0;
        uint32_t acc_row = 0;
        if constexpr (RULE == RULE_WEYL) {
            acc_row = weyl_const + p.weyl.mul_row * (row + (uint32_t)p.row_off0 + b * p.row_skip);
        } else if constexpr (RULE != RULE_RTN) {
            flat0 = ((uint64_t)row + p.row_off0 + (uint64_t)b * p.row_skip) * N;
            if constexpr (RULE == RULE_SR_HASH) acc_row = (uint32_t)flat0 * kHashP1 + ((uint32_t)(flat0 >> 32) ^ key1) * kHashP5 + hash_base;
        }
        uint4* sp = reinterpret_cast<uint4*>(state_w + (uint64_t)row * (CH * 16u));
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const uint64_t g = (flat0 + (uint64_t)c * EPL) >> 2;
            uint32_t acc0 = acc_row;
            if constexpr (RULE == RULE_WEYL) acc0 = acc_row + (uint32_t)(c * EPL) * p.weyl.mul_col;
            if constexpr (RULE == RULE_SR_HASH) acc0 = acc_row + (uint32_t)(c * EPL) * kHashP1;
            const uint4 packed = round_pack_lane<FMT, RULE>(v + c * EPL, acc0, p.weyl.mul_col, (uint32_t)g, (uint32_t)(g >> 32), step_t, p.layer,
                                                            key0, key1, p.scale_top);
            if (active) sp[c] = packed;
        }
    };

    issue(b_first, std::integral_constant<int, 0>{});
    cp_async_commit();
    for (uint32_t b = b_first; b < b_last; b += 2) {
        row_step(b, std::integral_constant<int, 0>{});
        if (b + 1 < b_last) row_step(b + 1, std::integral_constant<int, 1>{});
    }
    cp_async_wait<0>();
}

// Shapes covered: N = 16, headdim 1, one decay per state, the plain signature, scale and dither blocks of 16.
template <int FMT, int RULE>
cudaError_t try_launch_mamba1(const UpdateParams& p, cudaStream_t stream, bool& launched) {
    launched = false;
    if constexpr (FMT != FMT_FP32) {
        const bool extras = p.dt_bias || p.dt_softplus || p.z || p.ngroups > 1;
        if (extras || p.N != 16u || p.P != 1u) return cudaSuccess;
        if (Fmt<FMT>::kScaled && p.scale_block != 16u) return cudaSuccess;
        if (RULE == RULE_WEYL && p.weyl.block != 16u) return cudaSuccess;
        UpdateParams q = p;
        const uint32_t tiles = (p.H + kThreads - 1) / kThreads;
        // enough CTAs to fill the device a few times over, each walking a run of sequences with its A rows in registers
        uint32_t chunks = (148u * 8u + tiles - 1) / tiles;
        if (chunks > p.B) chunks = p.B;
        if (chunks > 65535u) chunks = 65535u;
        q.rps = (p.B + chunks - 1) / chunks;
        chunks = (p.B + q.rps - 1) / q.rps;
        launched = true;
        note_kernel(4);
        if (p.prepare_only) return cudaSuccess;
        return launch_update_kernel(ssd_update_mamba1_kernel<FMT, RULE>, dim3(tiles, chunks), 0, stream, q);
    }
    return cudaSuccess;
}

}  // namespace ssdq

// ssdq_stream.cuh -- the fused decode step as a persistent, software-pipelined kernel for the block-scaled
// one-byte stores (E4M3 and INTb with FP32 scales), where the work per byte moved is largest.
//
// Why a second kernel.  With one-byte codes a head's tile is only 8 KB and a CTA spends most of its life
// computing, so a kernel that loads its tile, computes and exits keeps too few bytes in flight to fill HBM
// (it ran at half the copy bandwidth with the issue slots half idle).  Here a CTA stays resident and walks a
// contiguous range of (b, h) items; the codes, x and scales of the next STAGES - 1 items are already on their way
// (cp.async into a ring of shared-memory stages, one commit group per item) while the current one is computed,
// so the memory system always has several tiles per CTA outstanding.  Each lane reads back only what it copied
// itself: cp.async.wait_group is the only synchronisation, there is no barrier and no wait on another thread.
//
// Arithmetic.  The same operations in the same order as ssd_update_tile_kernel (every stored bit is identical),
// issued two entries at a time with the packed binary32 instructions of sm_100 (mul/fma/add .f32x2, all rounding
// modes), the three-input max for the block maximum, a division by the format's constant that is exact by
// construction, and -- for the E4M3 dither -- Eq. 2 in integer form on the binary32 bits.
#pragma once
#include "ssdq_update.cuh"

#ifndef SSDQ_STREAM_STAGES
#define SSDQ_STREAM_STAGES 2
#endif
#ifndef SSDQ_STREAM_MINB
#define SSDQ_STREAM_MINB 4
#endif

namespace ssdq {

// Unpack one 32-bit word of one-byte codes into two packed pairs (exact widening).
__device__ __forceinline__ void unpack4_e4m3_x2(uint32_t w, f32x2& p01, f32x2& p23) {
    float f[4];
    unpack4_e4m3(w, f);
    p01 = pack2(f[0], f[1]);
    p23 = pack2(f[2], f[3]);
}
__device__ __forceinline__ void unpack4_int8_x2(uint32_t w, f32x2& p01, f32x2& p23) {
    w ^= 0x80808080u;                                      // bias to unsigned bytes
    const f32x2 off = pack2(-8388736.0f, -8388736.0f);     // -(2^23 + 128)
    p01 = add2_rn(pack2u(__byte_perm(w, 0x4B000000u, 0x7540), __byte_perm(w, 0x4B000000u, 0x7541)), off);
    p23 = add2_rn(pack2u(__byte_perm(w, 0x4B000000u, 0x7542), __byte_perm(w, 0x4B000000u, 0x7543)), off);
}

// Shared memory of one CTA: STAGES x { codes [RPS][kThreads] x 16 B, x [RPS/4][kThreads] x 16 B, scales [RPS/4][kThreads] x 16 B }.
template <int RPS, int STAGES>
constexpr size_t stream_smem_bytes() { return (size_t)STAGES * kThreads * 16u * (RPS + 2 * (RPS / 4)); }

// One-byte block-scaled stores, one decay per head, heads of P = (kThreads / LPR) * RPS rows, RPS a multiple of 4.
// ROW_SCALE: one scale per row of N entries (else one per 16 entries = per lane).
// grid = any number of CTAs <= n_items; CTA c owns items [c n / G, (c + 1) n / G).
template <int FMT, int RULE, int LPR, int RPS, int STAGES, bool ROW_SCALE>
__global__ void __launch_bounds__(kThreads, SSDQ_STREAM_MINB) ssd_update_stream_kernel(const UpdateParams p) {
    grid_dependency_gate(p.overlap);
    static_assert(Fmt<FMT>::kScaled && Fmt<FMT>::kEpl == 16, "one-byte block-scaled stores");
    static_assert(RPS % 4 == 0 && LPR >= 4 && STAGES >= 2, "rows are processed four at a time");
    constexpr int EPL = 16;
    constexpr int N = LPR * EPL;
    constexpr int NSLOT = kThreads / LPR;
    constexpr int ROWS = NSLOT * RPS;
    constexpr int SPR = ROW_SCALE ? 1 : N / 16;            // scales per row
    constexpr unsigned FULL = 0xFFFFFFFFu;
    constexpr uint32_t kTileStage = RPS * kThreads * 16u, kVecStage = (RPS / 4) * kThreads * 16u;

    extern __shared__ uint4 stream_smem[];
    const uint32_t tid = threadIdx.x;
    const uint32_t lis = tid % LPR;
    const uint32_t slot = tid / LPR;
    const uint32_t n0 = lis * EPL;
    // this lane's cell of every stage: byte addresses in the shared window
    const uint32_t tile_s = (uint32_t)__cvta_generic_to_shared(stream_smem) + tid * 16u;    // + stage * kTileStage + k * kThreads * 16
    const uint32_t x_s = tile_s + STAGES * kTileStage;                                       // + stage * kVecStage + k4 * kThreads * 16
    const uint32_t sc_s = x_s + STAGES * kVecStage;

    const uint32_t first = (uint32_t)(((uint64_t)blockIdx.x * p.n_items) / gridDim.x);
    const uint32_t last = (uint32_t)(((uint64_t)(blockIdx.x + 1) * p.n_items) / gridDim.x);
    if (first >= last) return;
    const uint32_t step_t = p.step_t + (p.step_base ? __ldcg(p.step_base) : 0u);
    const float top = p.scale_top, inv_top = p.inv_scale_top;

    // pointers of the item being fetched (f_*) and of the item being computed (c_*), advanced by one item per iteration
    const uint64_t row0 = (uint64_t)first * ROWS + slot * RPS;
    const uint4* f_codes = reinterpret_cast<const uint4*>(p.state) + row0 * LPR + lis;
    const float* f_x = p.x + row0;
    const float* f_sc = p.scales + row0 * SPR + (ROW_SCALE ? 0u : lis);
    uint4* c_codes = reinterpret_cast<uint4*>(p.state) + row0 * LPR + lis;
    float* c_sc = p.scales + row0 * SPR + (ROW_SCALE ? 0u : lis);
    float* c_y = p.y + row0 + lis / (LPR / 4);

    auto issue = [&](uint32_t stage) {
        // debug builds: the item's codes, x and scales must lie inside the caller's buffers (else nothing is copied)
        [[maybe_unused]] const uint64_t frow = (uint64_t)(f_x - p.x);
        bool mem_ok = SSDQ_RANGE_OK(p, DBG_STATE, frow * LPR + lis, (RPS - 1) * LPR + 1, state_vecs) && SSDQ_RANGE_OK(p, DBG_ROWS, frow, RPS, rows) &&
                      SSDQ_RANGE_OK(p, DBG_SCALES, frow * SPR + (ROW_SCALE ? 0u : lis), (RPS - 1) * SPR + 1, scales);
        if (mem_ok) {
#pragma unroll
        for (int k = 0; k < RPS; ++k) cp_async16(tile_s + stage * kTileStage + k * (kThreads * 16u), f_codes + k * LPR);
#pragma unroll
        for (int k4 = 0; k4 < RPS / 4; ++k4) {
            cp_async16_ca(x_s + stage * kVecStage + k4 * (kThreads * 16u), f_x + 4 * k4);
            const uint32_t sdst = sc_s + stage * kVecStage + k4 * (kThreads * 16u);
            if constexpr (ROW_SCALE) {
                cp_async16_ca(sdst, f_sc + 4 * k4);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) cp_async4_ca(sdst + 4 * j, f_sc + (4 * k4 + j) * SPR);
            }
        }
        }
        f_codes += ROWS * LPR;
        f_x += ROWS;
        f_sc += ROWS * SPR;
    };
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (first + s < last) issue(s);
        cp_async_commit();
    }

    LaneThreshold<FMT, RULE, LPR> thr;
    thr.init(p.weyl, step_t, lis);
    const uint32_t key0 = (uint32_t)p.sr_seed, key1 = (uint32_t)(p.sr_seed >> 32);
    const uint32_t hash_base = step_t * kHashP2 + p.layer * kHashP3 + key0 * kHashP4;
    const bool y_writer = (lis & (LPR / 4 - 1)) == 0;
    uint32_t b = first / p.H;
    uint32_t h = first - b * p.H;
    uint64_t grow_first = row0 + p.row_off0 + (uint64_t)b * p.row_skip;
    f32x2 B2[EPL / 2], C2[EPL / 2];
    // scalars of the next item are fetched one iteration ahead
    float dt_next = __ldg(p.dt + first), A_next = __ldg(p.A + h), D_next = (p.D && lis == 0) ? __ldg(p.D + h) : 0.0f;

    uint32_t stage = 0;
    uint32_t item = first;
    while (item < last) {
      // a run of items of one sequence b shares B and C
      {
        const float4* Bp = reinterpret_cast<const float4*>(p.Bm + (size_t)b * N + n0);
        const float4* Cp = reinterpret_cast<const float4*>(p.Cm + (size_t)b * N + n0);
        const bool bc_ok = SSDQ_RANGE_OK(p, DBG_BC, (size_t)b * N + n0, EPL, bc_floats);
#pragma unroll
        for (int i = 0; i < EPL / 4; ++i) {
            const float4 zero4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            const float4 bb = bc_ok ? __ldg(Bp + i) : zero4, cc = bc_ok ? __ldg(Cp + i) : zero4;
            B2[2 * i] = pack2(bb.x, bb.y); B2[2 * i + 1] = pack2(bb.z, bb.w);
            C2[2 * i] = pack2(cc.x, cc.y); C2[2 * i + 1] = pack2(cc.z, cc.w);
        }
      }
      const uint32_t run_end = min(last, (b + 1u) * p.H);
      for (; item < run_end; ++item) {
        // refill the stage that the previous iteration consumed
        {
            uint32_t fill = stage + (STAGES - 1);
            if (fill >= STAGES) fill -= STAGES;
            if (item + (STAGES - 1) < last) issue(fill);
            cp_async_commit();
        }
        const float dtv = dt_next, Dl = D_next;
        const float a = exp_spec(__fmul_rn(dtv, A_next));
        if (item + 1 < last && SSDQ_RANGE_OK(p, DBG_ITEMS, item + 1, 1, items)) {
            const uint32_t h_n = (h + 1u == p.H) ? 0u : h + 1u;
            dt_next = __ldg(p.dt + item + 1);
            A_next = __ldg(p.A + h_n);
            D_next = (p.D && lis == 0) ? __ldg(p.D + h_n) : 0.0f;
        }
        [[maybe_unused]] const uint64_t crow = (uint64_t)(c_y - p.y) - lis / (LPR / 4);
        const bool mem_ok = SSDQ_RANGE_OK(p, DBG_STATE, crow * LPR + lis, (RPS - 1) * LPR + 1, state_vecs) && SSDQ_RANGE_OK(p, DBG_ROWS, crow, RPS, rows) &&
                            SSDQ_RANGE_OK(p, DBG_SCALES, crow * SPR + (ROW_SCALE ? 0u : lis), (RPS - 1) * SPR + 1, scales);
        uint32_t acc_row = 0;
        uint64_t grp_row = 0;
        if constexpr (RULE == RULE_WEYL) acc_row = thr.weyl_acc0(grow_first);
        if constexpr (RULE == RULE_SR) grp_row = (grow_first * (uint64_t)N + n0) >> 2;
        const f32x2 a2 = pack2(a, a);

        cp_async_wait<STAGES - 1>();                  // this item's group has landed (later ones may be pending)
        // one row: dequantise, Eq. 1, partial dot, block scale, thresholds, Eq. 2, store; returns the lane's partial dot
        auto process_row = [&](const int k, const float xk, const float sk) -> float {
            uint32_t rw[4];
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(rw[0]), "=r"(rw[1]), "=r"(rw[2]), "=r"(rw[3]) : "r"(tile_s + stage * kTileStage + k * (kThreads * 16u)));
            f32x2 hv[EPL / 2];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if constexpr (FMT == FMT_E4M3) unpack4_e4m3_x2(rw[i], hv[2 * i], hv[2 * i + 1]);
                else unpack4_int8_x2(rw[i], hv[2 * i], hv[2 * i + 1]);
            }
            const float dtx = __fmul_rn(dtv, xk);
            const f32x2 dtx2 = pack2(dtx, dtx), sc2 = pack2(sk, sk);
            f32x2 dotA = pack2(__fmul_rn(Dl, xk), 0.0f), dotB = pack2(0.0f, 0.0f);
            float amaxA = 0.0f, amaxB = 0.0f;
#pragma unroll
            for (int i = 0; i < EPL / 2; i += 2) {
                const f32x2 Bi0 = B2[i], Bi1 = B2[i + 1], Ci0 = C2[i], Ci1 = C2[i + 1];
                const f32x2 hn0 = fma2_rn(a2, mul2_rn(hv[i], sc2), mul2_rn(dtx2, Bi0));
                const f32x2 hn1 = fma2_rn(a2, mul2_rn(hv[i + 1], sc2), mul2_rn(dtx2, Bi1));
                hv[i] = hn0;
                hv[i + 1] = hn1;
                dotA = fma2_rn(Ci0, hn0, dotA);
                dotB = fma2_rn(Ci1, hn1, dotB);
                float e0, e1, e2, e3;
                unpack2(hn0, e0, e1);
                unpack2(hn1, e2, e3);
                amaxA = max3abs(amaxA, e0, e1);
                amaxB = max3abs(amaxB, e2, e3);
            }
            float d0, d1;
            unpack2(add2_rn(dotA, dotB), d0, d1);
            float amax = fmaxf(amaxA, amaxB);
            if constexpr (ROW_SCALE) {
#pragma unroll
                for (int off = LPR / 2; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, off));
            }
            const float s = fmaxf(div_by_top(amax, top, inv_top), 1.17549435e-38f);
            const float rinv = rcp_scale(s);
            const f32x2 rinv2 = pack2(rinv, rinv);
            float v[EPL];
#pragma unroll
            for (int i = 0; i < EPL / 2; ++i) unpack2(mul2_rn(hv[i], rinv2), v[2 * i], v[2 * i + 1]);
            if constexpr (ROW_SCALE) { if (lis == 0 && mem_ok) c_sc[k] = s; }
            else if (mem_ok) c_sc[k * SPR] = s;

            uint32_t acc[EPL];
            if constexpr (RULE == RULE_WEYL) {
#pragma unroll
                for (int j = 0; j < EPL; ++j) acc[j] = acc_row + (uint32_t)j * p.weyl.mul_col;
                acc_row += thr.row_mul;
            } else if constexpr (RULE == RULE_SR_HASH) {
                const uint32_t key = thr.hash_key0(grow_first + k, hash_base, key1);
#pragma unroll
                for (int j = 0; j < EPL; ++j) acc[j] = fmix32(key + (uint32_t)j * kHashP1);
            } else if constexpr (RULE == RULE_SR) {
#pragma unroll
                for (int g = 0; g < EPL / 4; ++g) {
                    const uint4 o = philox4x32_10(make_uint4((uint32_t)grp_row + (uint32_t)g, (uint32_t)(grp_row >> 32), step_t, p.layer), key0, key1);
                    acc[4 * g] = o.x; acc[4 * g + 1] = o.y; acc[4 * g + 2] = o.z; acc[4 * g + 3] = o.w;
                }
                grp_row += N / 4;
            }
            if (mem_ok) c_codes[k * LPR] = round_pack16<FMT, RULE>(v, acc, top);
            return __fadd_rn(d0, d1);
        };
#pragma unroll
        for (int g4 = 0; g4 < RPS / 4; ++g4) {
            float4 x4, s4;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(x4.x), "=f"(x4.y), "=f"(x4.z), "=f"(x4.w) : "r"(x_s + stage * kVecStage + g4 * (kThreads * 16u)));
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(s4.x), "=f"(s4.y), "=f"(s4.z), "=f"(s4.w) : "r"(sc_s + stage * kVecStage + g4 * (kThreads * 16u)));
            const float d0 = process_row(g4 * 4 + 0, x4.x, s4.x);
            const float d1 = process_row(g4 * 4 + 1, x4.y, s4.y);
            const float d2 = process_row(g4 * 4 + 2, x4.z, s4.z);
            const float d3 = process_row(g4 * 4 + 3, x4.w, s4.w);
            const float tot = reduce4_over_slot<LPR>(d0, d1, d2, d3, lis);
            if (y_writer && mem_ok) c_y[g4 * 4] = tot;
        }
        c_codes += ROWS * LPR;
        c_sc += ROWS * SPR;
        c_y += ROWS;
        grow_first += ROWS;
        ++h;
        if (++stage == STAGES) stage = 0;
      }
      h = 0;
      ++b;
      grow_first += p.row_skip;       // over the rows that other head shards hold
    }
    cp_async_wait<0>();
}

// ---- host side --------------------------------------------------------------------------------------------------
// Resident CTAs per SM of one instantiation on the current device, and the device's SM count (queried once each).
template <int FMT, int RULE, int LPR, int RPS, int STAGES, bool ROW_SCALE>
inline cudaError_t stream_geometry(int& ctas_per_sm, int& sms) {
    constexpr int kMaxDevices = 64;
    static int cached_ctas[kMaxDevices] = {}, cached_sms[kMaxDevices] = {};     // per device; a race only repeats the queries
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (cached_ctas[dev] == 0) {
        auto kernel = ssd_update_stream_kernel<FMT, RULE, LPR, RPS, STAGES, ROW_SCALE>;
        constexpr size_t smem = stream_smem_bytes<RPS, STAGES>();
        if ((e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        int n = 0, occ = 0;
        if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kThreads, smem)) != cudaSuccess) return e;
        if (occ < 1 || n < 1) return cudaErrorInvalidConfiguration;
        cached_sms[dev] = n;
        cached_ctas[dev] = occ;
    }
    ctas_per_sm = cached_ctas[dev];
    sms = cached_sms[dev];
    return cudaSuccess;
}

template <int FMT, int RULE, int LPR, int RPS, int STAGES, bool ROW_SCALE>
inline cudaError_t launch_stream(const UpdateParams& p, cudaStream_t stream) {
    int ctas = 0, sms = 0;
    const cudaError_t e = stream_geometry<FMT, RULE, LPR, RPS, STAGES, ROW_SCALE>(ctas, sms);
    if (e != cudaSuccess) return e;
    uint32_t grid = (uint32_t)(ctas * sms);            // one wave of resident CTAs
    if (grid > p.n_items) grid = p.n_items;
    note_kernel(2);
    if (p.prepare_only) return cudaSuccess;
    return launch_update_kernel(ssd_update_stream_kernel<FMT, RULE, LPR, RPS, STAGES, ROW_SCALE>, dim3(grid), stream_smem_bytes<RPS, STAGES>(), stream, p);
}

// Shapes covered: N = 128 with heads of 64 or 128 rows, the plain signature (no dt_bias / softplus / groups / gate),
// x, y and the scales 16-byte aligned.  Two stages: one item in flight per CTA besides the one being computed was
// the fastest setting measured (a third stage was slower at every occupancy tried).
template <int FMT, int RULE, int LPR>
cudaError_t try_launch_stream(const UpdateParams& p, cudaStream_t stream, bool& launched) {
    launched = false;
    if constexpr (LPR == 8) {
        const bool extras = p.dt_bias || p.dt_softplus || p.z || p.ngroups > 1;
        const bool aligned = ((reinterpret_cast<uintptr_t>(p.x) | reinterpret_cast<uintptr_t>(p.y) | reinterpret_cast<uintptr_t>(p.scales)) & 15u) == 0;
        constexpr uint32_t nslot = kThreads / LPR;
        if (extras || !aligned || !(p.P == nslot * 4u || p.P == nslot * 8u)) return cudaSuccess;
        launched = true;
        const bool row_scale = p.scale_block == (uint32_t)(LPR * 16);
        if (p.P == nslot * 4u)
            return row_scale ? launch_stream<FMT, RULE, LPR, 4, SSDQ_STREAM_STAGES, true>(p, stream) : launch_stream<FMT, RULE, LPR, 4, SSDQ_STREAM_STAGES, false>(p, stream);
        return row_scale ? launch_stream<FMT, RULE, LPR, 8, SSDQ_STREAM_STAGES, true>(p, stream) : launch_stream<FMT, RULE, LPR, 8, SSDQ_STREAM_STAGES, false>(p, stream);
    }
    return cudaSuccess;
}

}  // namespace ssdq

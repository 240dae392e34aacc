// ssdq_api.cu -- the C ABI declared in include/ssdq.h: argument checks, then one launch per call
// (one per layer and step for the multi-step driver).  No device allocation, no global state
// besides a thread-local error text and a launch counter.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/ssdq.h"
#include "ssdq_internal.h"

namespace {

thread_local char g_err[256] = "";
std::atomic<uint64_t> g_launches{0};
std::atomic<int> g_launch_overlap{1};      // programmatic dependent launch between the drivers' own kernels

ssdq_status fail(ssdq_status code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

ssdq_status cuda_result(cudaError_t e, const char* what) {
    if (e == cudaSuccess) { g_launches.fetch_add(1, std::memory_order_relaxed); return SSDQ_OK; }
    return fail(SSDQ_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

bool format_known(int fmt) { return fmt >= SSDQ_FP16 && fmt <= SSDQ_INT4; }
bool format_scaled(int fmt) { return fmt == SSDQ_E4M3 || (fmt >= SSDQ_INT8 && fmt <= SSDQ_INT4); }
// kernel family of a public format id, and the top of its scaled range (amax maps onto it)
int kernel_format(int fmt) { return fmt >= SSDQ_INT8 ? (int)ssdq::FMT_INT : fmt; }
float scale_top(int fmt) {
    switch (fmt) {
        case SSDQ_E4M3: return 448.0f;
        case SSDQ_INT8: return 127.0f;
        case SSDQ_INT7: return 63.0f;
        case SSDQ_INT6: return 31.0f;
        case SSDQ_INT4: return 7.0f;
        default: return 1.0f;
    }
}

bool dstate_supported(int fmt, uint32_t n) {
    if (!(n == 16 || n == 32 || n == 64 || n == 128 || n == 256)) return false;
    if (fmt == SSDQ_FP32 && n > 128) return false;   // a row of 256 floats would span two warps
    return true;
}

ssdq::WeylConst weyl_const(const ssdq_weyl& w) {
    return ssdq::WeylConst{w.mul_row, w.mul_col, w.phi, w.base, w.block};
}

// Checks shared by ssd_state_update and ssd_decode_run; per-step pointers are checked separately.
ssdq_status check_layer(const ssdq_update_desc* d) {
    if (!d) return fail(SSDQ_ERR_NULL, "descriptor is NULL");
    if (d->batch == 0 || d->nheads == 0 || d->headdim == 0) return fail(SSDQ_ERR_SHAPE, "batch, nheads and headdim must be positive");
    if (!format_known(d->format)) return fail(SSDQ_ERR_UNSUPPORTED, "unknown format %d", d->format);
    if (d->rule < SSDQ_RTN || d->rule > SSDQ_SR_HASH) return fail(SSDQ_ERR_UNSUPPORTED, "unknown rule %d", d->rule);
    if (!dstate_supported(d->format, d->dstate)) return fail(SSDQ_ERR_UNSUPPORTED, "dstate %u is not supported for format %d", d->dstate, d->format);
    if ((uint64_t)d->batch * d->nheads > 0xFFFFFFFFull / 2) return fail(SSDQ_ERR_SHAPE, "batch * nheads too large");
    if (!d->state || !d->A) return fail(SSDQ_ERR_NULL, "state and A are required");
    if (!aligned16(d->state)) return fail(SSDQ_ERR_ALIGN, "state must be 16-byte aligned");
    if (d->a_per_state ? !aligned16(d->A) : !aligned4(d->A)) return fail(SSDQ_ERR_ALIGN, "A is misaligned");
    if (d->D && !aligned4(d->D)) return fail(SSDQ_ERR_ALIGN, "D is misaligned");
    if (d->dt_bias && !aligned4(d->dt_bias)) return fail(SSDQ_ERR_ALIGN, "dt_bias is misaligned");
    if (d->ngroups > 1 && d->nheads % d->ngroups != 0) return fail(SSDQ_ERR_SHAPE, "nheads must be a multiple of ngroups");
    if (d->nheads_global == 0 ? d->head_index_base != 0
                              : (d->nheads_global < d->nheads || d->head_index_base > d->nheads_global - d->nheads))
        return fail(SSDQ_ERR_SHAPE, "head shard [%u, %u + %u) does not fit in nheads_global = %u", d->head_index_base, d->head_index_base,
                    d->nheads, d->nheads_global);
    if ((uint64_t)(d->nheads_global ? d->nheads_global - d->nheads : 0u) * d->headdim > 0xFFFFFFFFull)
        return fail(SSDQ_ERR_SHAPE, "nheads_global * headdim is too large");
    if (format_scaled(d->format)) {
        if (!d->scales) return fail(SSDQ_ERR_NULL, "E4M3 and INTb stores need a scale array");
        if (!aligned4(d->scales)) return fail(SSDQ_ERR_ALIGN, "scales are misaligned");
        const bool head_scale = d->scale_block == (uint32_t)d->headdim * d->dstate && d->scale_block != d->dstate;
        if (head_scale) {
            // one scale per (sequence, head): heads of (128 / lanes per row) * {2, 4, 8} rows, one decay per head, plain signature
            const uint32_t lpr = d->dstate / 16u, rows = d->headdim * lpr;      // rows * 16 entries per lane set
            const bool shape_ok = lpr >= 4 && lpr <= 16 && (rows == 128u * 2u || rows == 128u * 4u || rows == 128u * 8u);
            if (!shape_ok || d->a_per_state || d->dt_bias || d->dt_softplus || d->z || d->ngroups > 1 || d->batch > 65535u)
                return fail(SSDQ_ERR_UNSUPPORTED, "one scale per head (scale_block = headdim * dstate) is built for dstate 64..256, "
                                                  "headdim * dstate / 2048 in {2, 4, 8}, one decay per head and the plain signature");
        } else if (!(d->scale_block == 16 || d->scale_block == d->dstate)) {
            return fail(SSDQ_ERR_SHAPE, "scale_block must be 16, dstate, or headdim * dstate");
        }
    }
    if (d->rule == SSDQ_WEYL && d->format != SSDQ_FP32) {
        if (!(d->weyl.block == 16 || d->weyl.block == d->dstate)) return fail(SSDQ_ERR_SHAPE, "weyl.block must be 16 or dstate");
        if (d->weyl.phi == 0 || (d->weyl.phi & 1u) == 0) return fail(SSDQ_ERR_SHAPE, "weyl descriptor is not initialised");
    }
    return SSDQ_OK;
}

ssdq_status check_step_ptrs(const float* x, const float* dt, const float* Bm, const float* Cm, const float* y, const float* z = nullptr) {
    if (!x || !dt || !Bm || !Cm || !y) return fail(SSDQ_ERR_NULL, "x, dt, Bm, Cm and y are required");
    if (!aligned4(x) || !aligned4(dt) || !aligned4(y) || !aligned4(z)) return fail(SSDQ_ERR_ALIGN, "x, dt, y or z is misaligned");
    if (!aligned16(Bm) || !aligned16(Cm)) return fail(SSDQ_ERR_ALIGN, "Bm and Cm must be 16-byte aligned");
    return SSDQ_OK;
}

#ifdef SSDQ_DEBUG
// The status words of the bounds-checking build: code of the first violation (0 = none), the offending index (low, high)
// and the block that saw it.
__device__ uint32_t g_debug_status[4];
uint32_t* debug_status_address() {
    static uint32_t* cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cached[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_debug_status) != cudaSuccess) return nullptr;
        cached[dev] = static_cast<uint32_t*>(ptr);
    }
    return cached[dev];
}
#endif

ssdq::UpdateParams make_params(const ssdq_update_desc* d, uint32_t step_t) {
    ssdq::UpdateParams p{};
    p.state = d->state; p.scales = d->scales;
    p.x = d->x; p.dt = d->dt; p.A = d->A; p.Bm = d->Bm; p.Cm = d->Cm; p.D = d->D; p.y = d->y;
    p.dt_bias = d->dt_bias; p.z = d->z; p.dt_softplus = d->dt_softplus;
    p.ngroups = d->ngroups > 1 ? d->ngroups : 1;
    p.heads_per_group = d->nheads / p.ngroups;
    p.B = d->batch; p.H = d->nheads; p.P = d->headdim; p.N = d->dstate;
    p.n_items = d->batch * d->nheads;
    p.scale_block = d->scale_block;
    p.scale_top = scale_top(d->format);
    p.inv_scale_top = 1.0f / p.scale_top;
    p.step_t = step_t; p.layer = d->layer;
    {
        const uint32_t Hg = d->nheads_global ? d->nheads_global : d->nheads;
        p.row_off0 = ((uint64_t)d->batch_index_base * Hg + d->head_index_base) * d->headdim;
        p.row_skip = (Hg - d->nheads) * d->headdim;
    }
    p.weyl = weyl_const(d->weyl);
    p.sr_seed = d->sr_seed;
#ifdef SSDQ_DEBUG
    {
        const uint64_t rows = (uint64_t)d->batch * d->nheads * d->headdim, entries = rows * d->dstate;
        const uint64_t bytes = d->format == SSDQ_FP32 ? 4u : (d->format == SSDQ_FP16 || d->format == SSDQ_BF16) ? 2u : 1u;
        p.dbg.status = debug_status_address();
        p.dbg.state_vecs = entries * bytes / 16u;
        p.dbg.rows = rows;
        p.dbg.scales = format_scaled(d->format) && d->scale_block ? entries / d->scale_block : 0u;
        p.dbg.items = (uint64_t)d->batch * d->nheads;
        p.dbg.bc_floats = (uint64_t)d->batch * p.ngroups * d->dstate;
    }
#endif
    return p;
}

cudaError_t launch_update(const ssdq::UpdateParams& p, int fmt, int rule, bool aps, cudaStream_t s) {
    switch (fmt) {
        case SSDQ_FP16: return ssdq::launch_update_fp16(p, rule, aps, s);
        case SSDQ_BF16: return ssdq::launch_update_bf16(p, rule, aps, s);
        case SSDQ_E4M3: return ssdq::launch_update_e4m3(p, rule, aps, s);
        case SSDQ_FP32: return ssdq::launch_update_fp32(p, rule, aps, s);
        case SSDQ_INT8: case SSDQ_INT7: case SSDQ_INT6: case SSDQ_INT4: return ssdq::launch_update_int8(p, rule, aps, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

namespace {

// Host-side resources of the host-buffer driver, one set per device: two copy streams and the events that
// chain copy-in -> compute -> copy-out per staging slot.  Created on first use; no device memory.
constexpr uint32_t kMaxStagingSlots = 8;
struct HostPipe {
    std::mutex mutex;
    bool ready = false;
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t start = nullptr;
    cudaEvent_t loaded[kMaxStagingSlots] = {}, computed[kMaxStagingSlots] = {}, stored[kMaxStagingSlots] = {};
};
HostPipe g_pipes[64];
std::mutex g_pipes_mutex;

ssdq_status host_pipe_for_current_device(HostPipe** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(SSDQ_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return fail(SSDQ_ERR_UNSUPPORTED, "device ordinal %d beyond the table", dev);
    std::lock_guard<std::mutex> lock(g_pipes_mutex);
    HostPipe& hp = g_pipes[dev];
    if (!hp.ready) {
        if ((e = cudaStreamCreateWithFlags(&hp.h2d, cudaStreamNonBlocking)) != cudaSuccess ||
            (e = cudaStreamCreateWithFlags(&hp.d2h, cudaStreamNonBlocking)) != cudaSuccess ||
            (e = cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming)) != cudaSuccess)
            return fail(SSDQ_ERR_CUDA, "stream/event creation: %s", cudaGetErrorString(e));
        for (uint32_t i = 0; i < kMaxStagingSlots; ++i)
            if ((e = cudaEventCreateWithFlags(&hp.loaded[i], cudaEventDisableTiming)) != cudaSuccess ||
                (e = cudaEventCreateWithFlags(&hp.computed[i], cudaEventDisableTiming)) != cudaSuccess ||
                (e = cudaEventCreateWithFlags(&hp.stored[i], cudaEventDisableTiming)) != cudaSuccess)
                return fail(SSDQ_ERR_CUDA, "event creation: %s", cudaGetErrorString(e));
        hp.ready = true;
    }
    *out = &hp;
    return SSDQ_OK;
}

}  // namespace

namespace {
thread_local int g_last_kernel = -1;
}
namespace ssdq {
void note_kernel(int family) { g_last_kernel = family; }
int report_failure(int status, const char* text) { return fail(static_cast<ssdq_status>(status), "%s", text); }
void count_launches(unsigned n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
}  // namespace ssdq

extern "C" {

ssdq_status weyl_offsets_init(ssdq_weyl* out, uint32_t layer, uint32_t seed, uint32_t block) {
    if (!out) return fail(SSDQ_ERR_NULL, "out is NULL");
    if (block == 0 || block % 16 != 0) return fail(SSDQ_ERR_SHAPE, "block must be a positive multiple of 16");
    // Appendix B "Dithers": the decimal generators times 2^32, rounded to the nearest integer.
    const uint32_t kRow = 3242174889u, kCol = 2447445414u, kLayer = 530242489u, kSeed = 1349303490u;
    out->mul_row = kRow;
    out->mul_col = kCol;
    out->phi = 2654435769u;
    out->base = kLayer * layer + kSeed * seed;
    out->block = block;
    out->layer = layer;
    out->seed = seed;
    out->reserved = 0;
    g_err[0] = 0;
    return SSDQ_OK;
}

ssdq_status ssdq_thresholds_materialize(int rule, const ssdq_weyl* weyl, uint64_t sr_seed, uint32_t layer, uint64_t first_flat,
                                uint64_t n, uint32_t step_t, uint32_t* out_u24, void* stream) {
    if (rule < SSDQ_RTN || rule > SSDQ_SR_HASH) return fail(SSDQ_ERR_UNSUPPORTED, "unknown rule %d", rule);
    if (n && !out_u24) return fail(SSDQ_ERR_NULL, "out_u24 is NULL");
    ssdq::WeylConst w{};
    if (rule == SSDQ_WEYL) {
        if (!weyl) return fail(SSDQ_ERR_NULL, "weyl descriptor is NULL");
        if (weyl->block == 0) return fail(SSDQ_ERR_SHAPE, "weyl.block is zero");
        w = weyl_const(*weyl);
    }
    if (n == 0) return SSDQ_OK;
    return cuda_result(ssdq::launch_thresholds(rule, w, sr_seed, layer, first_flat, n, step_t, out_u24,
                                               static_cast<cudaStream_t>(stream)), "thresholds kernel");
}

ssdq_status ssd_state_update(const ssdq_update_desc* d, uint32_t step_t, void* stream) {
    ssdq_status rc = check_layer(d);
    if (rc != SSDQ_OK) return rc;
    rc = check_step_ptrs(d->x, d->dt, d->Bm, d->Cm, d->y, d->z);
    if (rc != SSDQ_OK) return rc;
    const ssdq::UpdateParams p = make_params(d, step_t);
    return cuda_result(launch_update(p, d->format, d->rule, d->a_per_state != 0, static_cast<cudaStream_t>(stream)),
                       "state-update kernel");
}

// quantize_store with the row mapping of a head shard: global row = row_index_base + row + (row / rows_per_seq) * row_skip
// (rows_per_seq == 0: rows are contiguous in the global view).
static ssdq_status quantize_rows(const float* src, void* dst_codes, float* dst_scales, uint64_t n_rows, uint32_t row_len,
                                 uint32_t scale_block, int format, int rule, const ssdq_weyl* weyl, uint64_t sr_seed, uint32_t layer,
                                 uint64_t row_index_base, uint64_t rows_per_seq, uint32_t row_skip, uint32_t step_t, void* stream) {
    if (!format_known(format)) return fail(SSDQ_ERR_UNSUPPORTED, "unknown format %d", format);
    if (rule < SSDQ_RTN || rule > SSDQ_SR_HASH) return fail(SSDQ_ERR_UNSUPPORTED, "unknown rule %d", rule);
    if (!dstate_supported(format, row_len)) return fail(SSDQ_ERR_UNSUPPORTED, "row_len %u is not supported for format %d", row_len, format);
    if (n_rows == 0) return SSDQ_OK;
    if (!src || !dst_codes) return fail(SSDQ_ERR_NULL, "src and dst_codes are required");
    if (!aligned16(src) || !aligned16(dst_codes)) return fail(SSDQ_ERR_ALIGN, "src and dst_codes must be 16-byte aligned");
    ssdq::QuantParams p{};
    if (format_scaled(format)) {
        if (!dst_scales) return fail(SSDQ_ERR_NULL, "E4M3 and INTb stores need a scale array");
        if (!(scale_block == 16 || scale_block == row_len)) return fail(SSDQ_ERR_SHAPE, "scale_block must be 16 or row_len");
    }
    if (rule == SSDQ_WEYL && format != SSDQ_FP32) {
        if (!weyl) return fail(SSDQ_ERR_NULL, "weyl descriptor is NULL");
        if (!(weyl->block == 16 || weyl->block == row_len)) return fail(SSDQ_ERR_SHAPE, "weyl.block must be 16 or row_len");
        p.weyl = weyl_const(*weyl);
    }
    p.src = src; p.codes = dst_codes; p.scales = dst_scales; p.n_rows = n_rows; p.row_len = row_len;
    p.scale_block = scale_block; p.scale_top = scale_top(format); p.step_t = step_t; p.layer = layer; p.row_base = row_index_base; p.sr_seed = sr_seed;
    p.rows_per_seq = row_skip ? rows_per_seq : 0; p.row_skip = row_skip;
    return cuda_result(ssdq::launch_quantize(p, kernel_format(format), rule, static_cast<cudaStream_t>(stream)), "quantize kernel");
}

ssdq_status quantize_store(const float* src, void* dst_codes, float* dst_scales, uint64_t n_rows, uint32_t row_len,
                   uint32_t scale_block, int format, int rule, const ssdq_weyl* weyl, uint64_t sr_seed, uint32_t layer,
                   uint64_t row_index_base, uint32_t step_t, void* stream) {
    return quantize_rows(src, dst_codes, dst_scales, n_rows, row_len, scale_block, format, rule, weyl, sr_seed, layer, row_index_base,
                         0, 0, step_t, stream);
}

ssdq_status ssd_replay_step(const float* w, const float* decay, uint32_t rows_per_decay, void* codes, float* scales, uint64_t n_rows,
                    uint32_t row_len, uint32_t scale_block, int format, int rule, const ssdq_weyl* weyl, uint64_t sr_seed,
                    uint32_t layer, uint64_t row_index_base, uint32_t step_t, void* stream) {
    if (!format_known(format)) return fail(SSDQ_ERR_UNSUPPORTED, "unknown format %d", format);
    if (rule < SSDQ_RTN || rule > SSDQ_SR_HASH) return fail(SSDQ_ERR_UNSUPPORTED, "unknown rule %d", rule);
    if (!dstate_supported(format, row_len)) return fail(SSDQ_ERR_UNSUPPORTED, "row_len %u is not supported for format %d", row_len, format);
    if (rows_per_decay == 0 || n_rows % rows_per_decay != 0) return fail(SSDQ_ERR_SHAPE, "n_rows must be a multiple of rows_per_decay");
    if (n_rows == 0) return SSDQ_OK;
    if (!w || !decay || !codes) return fail(SSDQ_ERR_NULL, "w, decay and codes are required");
    if (!aligned16(w) || !aligned16(codes) || !aligned4(decay)) return fail(SSDQ_ERR_ALIGN, "w and codes must be 16-byte aligned");
    ssdq::QuantParams p{};
    if (format_scaled(format)) {
        if (!scales) return fail(SSDQ_ERR_NULL, "E4M3 and INTb stores need a scale array");
        if (!(scale_block == 16 || scale_block == row_len)) return fail(SSDQ_ERR_SHAPE, "scale_block must be 16 or row_len");
    }
    if (rule == SSDQ_WEYL && format != SSDQ_FP32) {
        if (!weyl) return fail(SSDQ_ERR_NULL, "weyl descriptor is NULL");
        if (!(weyl->block == 16 || weyl->block == row_len)) return fail(SSDQ_ERR_SHAPE, "weyl.block must be 16 or row_len");
        p.weyl = weyl_const(*weyl);
    }
    p.src = w; p.decay = decay; p.rows_per_decay = rows_per_decay; p.codes = codes; p.scales = scales; p.n_rows = n_rows;
    p.row_len = row_len; p.scale_block = scale_block; p.scale_top = scale_top(format); p.step_t = step_t; p.layer = layer;
    p.row_base = row_index_base; p.sr_seed = sr_seed;
    return cuda_result(ssdq::launch_quantize(p, kernel_format(format), format == SSDQ_FP32 ? (int)SSDQ_RTN : rule,
                                             static_cast<cudaStream_t>(stream)), "replay kernel");
}

ssdq_status ssd_decode_run_checkpointed(const ssdq_update_desc* layers, float* const* work_fp32, uint32_t n_layers, uint32_t every,
                                uint32_t t_first, uint32_t n_steps, const ssdq_step_inputs* in, void* stream) {
    if (!layers || !in || !work_fp32) return fail(SSDQ_ERR_NULL, "layers, work_fp32 and in are required");
    if (n_layers == 0 || in->ring == 0 || every == 0) return fail(SSDQ_ERR_SHAPE, "n_layers, ring and every must be positive");
    for (uint32_t l = 0; l < n_layers; ++l) {
        const ssdq_status rc = check_layer(&layers[l]);
        if (rc != SSDQ_OK) return rc;
        if (layers[l].format == SSDQ_FP32) return fail(SSDQ_ERR_UNSUPPORTED, "the store of a checkpointed run must be a quantised format");
        if (!work_fp32[l] || !aligned16(work_fp32[l])) return fail(SSDQ_ERR_ALIGN, "work_fp32[l] must be a 16-byte aligned device buffer");
        if (layers[l].dstate > 128) return fail(SSDQ_ERR_UNSUPPORTED, "checkpointed runs need dstate <= 128 (FP32 working state)");
    }
    const uint32_t slots = n_steps < in->ring ? n_steps : in->ring;
    for (uint32_t sl = 0; sl < slots; ++sl)
        for (uint32_t l = 0; l < n_layers; ++l) {
            const uint64_t k = (uint64_t)sl * n_layers + l;
            const ssdq_status rc = check_step_ptrs(in->x + k * in->stride_x, in->dt + k * in->stride_dt, in->Bm + k * in->stride_B,
                                           in->Cm + k * in->stride_C, in->y + k * in->stride_y, in->z ? in->z + k * in->stride_z : nullptr);
            if (rc != SSDQ_OK) return rc;
        }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (uint32_t i = 0; i < n_steps; ++i) {
        const uint32_t t = t_first + i;
        for (uint32_t l = 0; l < n_layers; ++l) {
            const ssdq_update_desc& d = layers[l];
            const uint64_t k = (uint64_t)(i % in->ring) * n_layers + l;
            // the update itself runs on the FP32 working state, unrounded
            ssdq::UpdateParams p = make_params(&d, t);
            p.state = work_fp32[l]; p.scales = nullptr; p.scale_block = 0;
#ifdef SSDQ_DEBUG
            p.dbg.state_vecs = (uint64_t)d.batch * d.nheads * d.headdim * d.dstate / 4u;      // binary32 working state
            p.dbg.scales = 0;
#endif
            p.x = in->x + k * in->stride_x;
            p.dt = in->dt + k * in->stride_dt;
            p.Bm = in->Bm + k * in->stride_B;
            p.Cm = in->Cm + k * in->stride_C;
            p.y = in->y + k * in->stride_y;
            p.z = in->z ? in->z + k * in->stride_z : nullptr;
            p.overlap = (i | l) != 0 && g_launch_overlap.load(std::memory_order_relaxed) != 0;
            ssdq_status rc = cuda_result(launch_update(p, SSDQ_FP32, SSDQ_RTN, d.a_per_state != 0, s), "state-update kernel");
            if (rc != SSDQ_OK) return rc;
            if ((i + 1) % every != 0) continue;
            // every `every`-th write is rounded into the store (Eq. 2 under the layer's rule) and read back
            const uint64_t n_rows = (uint64_t)d.batch * d.nheads * d.headdim;
            const uint32_t Hg = d.nheads_global ? d.nheads_global : d.nheads;
            rc = quantize_rows(work_fp32[l], d.state, d.scales, n_rows, d.dstate, d.scale_block, d.format, d.rule, &d.weyl,
                               d.sr_seed, d.layer, ((uint64_t)d.batch_index_base * Hg + d.head_index_base) * d.headdim,
                               (uint64_t)d.nheads * d.headdim, (Hg - d.nheads) * d.headdim, t, stream);
            if (rc != SSDQ_OK) return rc;
            rc = ssdq_dequantize(d.state, d.scales, n_rows * d.dstate, d.format, d.scale_block, work_fp32[l], stream);
            if (rc != SSDQ_OK) return rc;
        }
    }
    return SSDQ_OK;
}

ssdq_status ssdq_dequantize(const void* codes, const float* scales, uint64_t n, int format, uint32_t scale_block, float* out,
                    void* stream) {
    if (!format_known(format)) return fail(SSDQ_ERR_UNSUPPORTED, "unknown format %d", format);
    if (n == 0) return SSDQ_OK;
    if (!codes || !out) return fail(SSDQ_ERR_NULL, "codes and out are required");
    if (n % 16 != 0) return fail(SSDQ_ERR_SHAPE, "n must be a multiple of 16");
    if (!aligned16(codes) || !aligned16(out)) return fail(SSDQ_ERR_ALIGN, "codes and out must be 16-byte aligned");
    if (format_scaled(format) && (!scales || scale_block == 0 || scale_block % 16 != 0))
        return fail(SSDQ_ERR_SHAPE, "scaled stores need scales and a scale_block that is a multiple of 16");
    return cuda_result(ssdq::launch_dequantize(codes, scales, n, kernel_format(format), scale_block, out, static_cast<cudaStream_t>(stream)),
                       "dequantize kernel");
}

ssdq_status ssd_decode_run(const ssdq_update_desc* layers, uint32_t n_layers, uint32_t t_first, uint32_t n_steps,
                   const ssdq_step_inputs* in, void* stream) {
    if (!layers || !in) return fail(SSDQ_ERR_NULL, "layers and in are required");
    if (n_layers == 0 || in->ring == 0) return fail(SSDQ_ERR_SHAPE, "n_layers and ring must be positive");
    for (uint32_t l = 0; l < n_layers; ++l) {
        const ssdq_status rc = check_layer(&layers[l]);
        if (rc != SSDQ_OK) return rc;
    }
    // every slot of the ring is used with every layer: check the alignment of each (slot, layer) once
    const uint32_t slots = n_steps < in->ring ? n_steps : in->ring;
    for (uint32_t s = 0; s < slots; ++s)
        for (uint32_t l = 0; l < n_layers; ++l) {
            const uint64_t k = (uint64_t)s * n_layers + l;
            const ssdq_status rc = check_step_ptrs(in->x + k * in->stride_x, in->dt + k * in->stride_dt, in->Bm + k * in->stride_B,
                                                   in->Cm + k * in->stride_C, in->y + k * in->stride_y, in->z ? in->z + k * in->stride_z : nullptr);
            if (rc != SSDQ_OK) return rc;
        }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (uint32_t i = 0; i < n_steps; ++i) {
        const uint32_t t = t_first + i;
        for (uint32_t l = 0; l < n_layers; ++l) {
            const uint64_t k = (uint64_t)(i % in->ring) * n_layers + l;
            ssdq::UpdateParams p = make_params(&layers[l], t);
            p.x = in->x + k * in->stride_x;
            p.dt = in->dt + k * in->stride_dt;
            p.Bm = in->Bm + k * in->stride_B;
            p.Cm = in->Cm + k * in->stride_C;
            p.y = in->y + k * in->stride_y;
            p.z = in->z ? in->z + k * in->stride_z : nullptr;
            p.overlap = (i | l) != 0 && g_launch_overlap.load(std::memory_order_relaxed) != 0;   // not after foreign work
            const ssdq_status rc = cuda_result(launch_update(p, layers[l].format, layers[l].rule, layers[l].a_per_state != 0, s),
                                       "state-update kernel");
            if (rc != SSDQ_OK) return rc;
        }
    }
    return SSDQ_OK;
}

uint64_t ssdq_state_error_workspace_bytes(uint32_t batch, uint32_t nheads) { return (uint64_t)batch * nheads * 16u; }

ssdq_status ssdq_state_error(const void* codes, const float* scales, const float* twin, uint32_t batch, uint32_t nheads,
                     uint32_t headdim, uint32_t dstate, int format, uint32_t scale_block, double* err2_per_head,
                     double* ref2_per_head, void* workspace, uint64_t workspace_bytes, void* stream) {
    if (!format_known(format)) return fail(SSDQ_ERR_UNSUPPORTED, "unknown format %d", format);
    if (batch == 0 || nheads == 0 || headdim == 0 || dstate == 0) return fail(SSDQ_ERR_SHAPE, "sizes must be positive");
    if (((uint64_t)headdim * dstate) % 16 != 0) return fail(SSDQ_ERR_SHAPE, "headdim * dstate must be a multiple of 16");
    if ((uint64_t)batch * nheads > 0x7FFFFFFFull) return fail(SSDQ_ERR_SHAPE, "batch * nheads too large");
    if (!codes || !twin || !err2_per_head || !ref2_per_head || !workspace) return fail(SSDQ_ERR_NULL, "codes, twin, outputs and workspace are required");
    if (!aligned16(codes) || !aligned16(workspace) || !aligned4(twin)) return fail(SSDQ_ERR_ALIGN, "codes and workspace must be 16-byte aligned");
    if (workspace_bytes < ssdq_state_error_workspace_bytes(batch, nheads)) return fail(SSDQ_ERR_SHAPE, "workspace too small");
    if (format_scaled(format) && (!scales || scale_block == 0 || scale_block % 16 != 0))
        return fail(SSDQ_ERR_SHAPE, "scaled stores need scales and a scale_block that is a multiple of 16");
    const ssdq_status rc = cuda_result(ssdq::launch_state_error(codes, scales, twin, batch, nheads, headdim * dstate, kernel_format(format), scale_block,
                                                        err2_per_head, ref2_per_head, workspace, static_cast<cudaStream_t>(stream)),
                               "state-error kernels");
    if (rc == SSDQ_OK) g_launches.fetch_add(1, std::memory_order_relaxed);   // two kernels per call
    return rc;
}

ssdq_status ssdq_readout_kl(const float* y_ref, const float* y_q, uint32_t batch, uint32_t width, float* kl_per_sequence, void* stream) {
    if (batch == 0 || width == 0) return fail(SSDQ_ERR_SHAPE, "batch and width must be positive");
    if (!y_ref || !y_q || !kl_per_sequence) return fail(SSDQ_ERR_NULL, "y_ref, y_q and kl_per_sequence are required");
    return cuda_result(ssdq::launch_readout_kl(y_ref, y_q, batch, width, kl_per_sequence, static_cast<cudaStream_t>(stream)),
                       "readout-KL kernel");
}

ssdq_status ssd_decode_run_host(const ssdq_update_desc* layers, uint32_t n_layers, uint32_t t_first, uint32_t n_steps,
                        const ssdq_step_inputs* host, const ssdq_step_inputs* staging, void* stream) {
    if (!layers || !host || !staging) return fail(SSDQ_ERR_NULL, "layers, host and staging are required");
    if (n_layers == 0 || host->ring == 0) return fail(SSDQ_ERR_SHAPE, "n_layers and host ring must be positive");
    if (staging->ring < 2 || staging->ring > kMaxStagingSlots) return fail(SSDQ_ERR_SHAPE, "staging ring must hold 2 to 8 slots");
    if (host->stride_x != staging->stride_x || host->stride_dt != staging->stride_dt || host->stride_B != staging->stride_B ||
        host->stride_C != staging->stride_C || host->stride_y != staging->stride_y || host->stride_z != staging->stride_z ||
        (host->z == nullptr) != (staging->z == nullptr))
        return fail(SSDQ_ERR_SHAPE, "host and staging strides must be equal");
    if (!host->x || !host->dt || !host->Bm || !host->Cm || !host->y) return fail(SSDQ_ERR_NULL, "host x, dt, Bm, Cm and y are required");
    if (!aligned4(host->x) || !aligned4(host->dt) || !aligned4(host->Bm) || !aligned4(host->Cm) || !aligned4(host->y) || !aligned4(host->z))
        return fail(SSDQ_ERR_ALIGN, "host arrays must be 4-byte aligned");
    for (uint32_t l = 0; l < n_layers; ++l) {
        const ssdq_status rc = check_layer(&layers[l]);
        if (rc != SSDQ_OK) return rc;
    }
    for (uint32_t sl = 0; sl < staging->ring; ++sl)
        for (uint32_t l = 0; l < n_layers; ++l) {
            const uint64_t k = (uint64_t)sl * n_layers + l;
            const ssdq_status rc = check_step_ptrs(staging->x + k * staging->stride_x, staging->dt + k * staging->stride_dt,
                                           staging->Bm + k * staging->stride_B, staging->Cm + k * staging->stride_C,
                                           staging->y + k * staging->stride_y, staging->z ? staging->z + k * staging->stride_z : nullptr);
            if (rc != SSDQ_OK) return rc;
        }
    if (n_steps == 0) return SSDQ_OK;
    cudaStream_t compute = static_cast<cudaStream_t>(stream);
    HostPipe* hp = nullptr;
    ssdq_status rc = host_pipe_for_current_device(&hp);
    if (rc != SSDQ_OK) return rc;
    std::lock_guard<std::mutex> lock(hp->mutex);
#define SSDQ_TRY(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail(SSDQ_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); } while (0)
    // staging slots may still be read by earlier work on the caller's stream
    SSDQ_TRY(cudaEventRecord(hp->start, compute));
    SSDQ_TRY(cudaStreamWaitEvent(hp->h2d, hp->start, 0));
    const uint32_t S = staging->ring;
    const uint64_t L = n_layers;
    for (uint32_t i = 0; i < n_steps; ++i) {
        const uint32_t sl = i % S;
        const uint64_t hk = (uint64_t)(i % host->ring) * L, dk = (uint64_t)sl * L;
        // inputs of step i: host slot -> staging slot, once the launches that last used the slot are done
        if (i >= S) SSDQ_TRY(cudaStreamWaitEvent(hp->h2d, hp->computed[sl], 0));
        SSDQ_TRY(cudaMemcpyAsync(const_cast<float*>(staging->x) + dk * staging->stride_x, host->x + hk * host->stride_x,
                                 L * host->stride_x * sizeof(float), cudaMemcpyHostToDevice, hp->h2d));
        SSDQ_TRY(cudaMemcpyAsync(const_cast<float*>(staging->dt) + dk * staging->stride_dt, host->dt + hk * host->stride_dt,
                                 L * host->stride_dt * sizeof(float), cudaMemcpyHostToDevice, hp->h2d));
        SSDQ_TRY(cudaMemcpyAsync(const_cast<float*>(staging->Bm) + dk * staging->stride_B, host->Bm + hk * host->stride_B,
                                 L * host->stride_B * sizeof(float), cudaMemcpyHostToDevice, hp->h2d));
        SSDQ_TRY(cudaMemcpyAsync(const_cast<float*>(staging->Cm) + dk * staging->stride_C, host->Cm + hk * host->stride_C,
                                 L * host->stride_C * sizeof(float), cudaMemcpyHostToDevice, hp->h2d));
        if (host->z)
            SSDQ_TRY(cudaMemcpyAsync(const_cast<float*>(staging->z) + dk * staging->stride_z, host->z + hk * host->stride_z,
                                     L * host->stride_z * sizeof(float), cudaMemcpyHostToDevice, hp->h2d));
        SSDQ_TRY(cudaEventRecord(hp->loaded[sl], hp->h2d));
        // the fused updates of step i, once its inputs have landed and the slot's previous y has left
        SSDQ_TRY(cudaStreamWaitEvent(compute, hp->loaded[sl], 0));
        if (i >= S) SSDQ_TRY(cudaStreamWaitEvent(compute, hp->stored[sl], 0));
        for (uint32_t l = 0; l < n_layers; ++l) {
            const uint64_t k = dk + l;
            ssdq::UpdateParams p = make_params(&layers[l], t_first + i);
            p.x = staging->x + k * staging->stride_x;
            p.dt = staging->dt + k * staging->stride_dt;
            p.Bm = staging->Bm + k * staging->stride_B;
            p.Cm = staging->Cm + k * staging->stride_C;
            p.y = staging->y + k * staging->stride_y;
            p.z = staging->z ? staging->z + k * staging->stride_z : nullptr;
            p.overlap = 0;      // measured: beside the two copy streams the attribute costs 14 % per step instead of gaining
            rc = cuda_result(launch_update(p, layers[l].format, layers[l].rule, layers[l].a_per_state != 0, compute),
                             "state-update kernel");
            if (rc != SSDQ_OK) return rc;
        }
        SSDQ_TRY(cudaEventRecord(hp->computed[sl], compute));
        // y of step i back to the host
        SSDQ_TRY(cudaStreamWaitEvent(hp->d2h, hp->computed[sl], 0));
        SSDQ_TRY(cudaMemcpyAsync(host->y + hk * host->stride_y, staging->y + dk * staging->stride_y,
                                 L * host->stride_y * sizeof(float), cudaMemcpyDeviceToHost, hp->d2h));
        SSDQ_TRY(cudaEventRecord(hp->stored[sl], hp->d2h));
    }
    // the caller's stream is complete only when every y has reached the host
    const uint32_t used = n_steps < S ? n_steps : S;
    for (uint32_t sl = 0; sl < used; ++sl) SSDQ_TRY(cudaStreamWaitEvent(compute, hp->stored[sl], 0));
#undef SSDQ_TRY
    return SSDQ_OK;
}

struct ssdq_graph {
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    uint32_t steps = 0, n_layers = 0;
};

ssdq_status ssd_decode_graph_create(ssdq_graph** out, const ssdq_update_desc* layers, uint32_t n_layers, uint32_t steps_per_launch,
                            const ssdq_step_inputs* in, uint32_t* step_counter) {
    if (!out || !layers || !in || !step_counter) return fail(SSDQ_ERR_NULL, "out, layers, in and step_counter are required");
    *out = nullptr;
    if (n_layers == 0 || in->ring == 0 || steps_per_launch == 0) return fail(SSDQ_ERR_SHAPE, "n_layers, ring and steps_per_launch must be positive");
    if (steps_per_launch % in->ring != 0) return fail(SSDQ_ERR_SHAPE, "steps_per_launch must be a multiple of the input ring");
    if (!aligned4(step_counter)) return fail(SSDQ_ERR_ALIGN, "step_counter is misaligned");
    for (uint32_t l = 0; l < n_layers; ++l) {
        const ssdq_status rc = check_layer(&layers[l]);
        if (rc != SSDQ_OK) return rc;
    }
    for (uint32_t sl = 0; sl < in->ring; ++sl)
        for (uint32_t l = 0; l < n_layers; ++l) {
            const uint64_t k = (uint64_t)sl * n_layers + l;
            const ssdq_status rc = check_step_ptrs(in->x + k * in->stride_x, in->dt + k * in->stride_dt, in->Bm + k * in->stride_B,
                                           in->Cm + k * in->stride_C, in->y + k * in->stride_y, in->z ? in->z + k * in->stride_z : nullptr);
            if (rc != SSDQ_OK) return rc;
        }
    // one-time set-up of the kernels the layers will use (function attributes, occupancy queries) happens here, before the
    // capture: nothing but launches is issued while the stream is capturing
    for (uint32_t l = 0; l < n_layers; ++l) {
        ssdq::UpdateParams p = make_params(&layers[l], 1u);
        p.x = in->x; p.y = in->y; p.z = in->z;
        p.prepare_only = 1;
        const cudaError_t pe = launch_update(p, layers[l].format, layers[l].rule, layers[l].a_per_state != 0, nullptr);
        if (pe != cudaSuccess) return fail(SSDQ_ERR_CUDA, "state-update kernel set-up: %s", cudaGetErrorString(pe));
    }
    cudaStream_t cs = nullptr;
    cudaError_t e = cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking);
    if (e != cudaSuccess) return fail(SSDQ_ERR_CUDA, "cudaStreamCreate: %s", cudaGetErrorString(e));
    ssdq_graph* g = new ssdq_graph();
    g->steps = steps_per_launch;
    g->n_layers = n_layers;
    ssdq_status rc = SSDQ_OK;
    e = cudaStreamBeginCapture(cs, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) rc = fail(SSDQ_ERR_CUDA, "cudaStreamBeginCapture: %s", cudaGetErrorString(e));
    if (rc == SSDQ_OK) {
        for (uint32_t i = 0; i < steps_per_launch && rc == SSDQ_OK; ++i)
            for (uint32_t l = 0; l < n_layers && rc == SSDQ_OK; ++l) {
                const uint64_t k = (uint64_t)(i % in->ring) * n_layers + l;
                ssdq::UpdateParams p = make_params(&layers[l], 1u + i);     // write index = counter + 1 + i
                p.step_base = step_counter;
                p.x = in->x + k * in->stride_x;
                p.dt = in->dt + k * in->stride_dt;
                p.Bm = in->Bm + k * in->stride_B;
                p.Cm = in->Cm + k * in->stride_C;
                p.y = in->y + k * in->stride_y;
                p.z = in->z ? in->z + k * in->stride_z : nullptr;
                p.overlap = 0;      // measured: kernel nodes joined by programmatic edges replay at half the rate of plain edges
                const cudaError_t le = launch_update(p, layers[l].format, layers[l].rule, layers[l].a_per_state != 0, cs);
                if (le != cudaSuccess) rc = fail(SSDQ_ERR_CUDA, "state-update kernel (capture): %s", cudaGetErrorString(le));
            }
        if (rc == SSDQ_OK) {
            const cudaError_t le = ssdq::launch_counter_add(step_counter, steps_per_launch, cs);
            if (le != cudaSuccess) rc = fail(SSDQ_ERR_CUDA, "counter kernel (capture): %s", cudaGetErrorString(le));
        }
        e = cudaStreamEndCapture(cs, &g->graph);         // always end the capture, also after a failed launch
        if (rc == SSDQ_OK && e != cudaSuccess) rc = fail(SSDQ_ERR_CUDA, "cudaStreamEndCapture: %s", cudaGetErrorString(e));
    }
    if (rc == SSDQ_OK) {
        e = cudaGraphInstantiate(&g->exec, g->graph, 0);
        if (e != cudaSuccess) rc = fail(SSDQ_ERR_CUDA, "cudaGraphInstantiate: %s", cudaGetErrorString(e));
    }
    cudaStreamDestroy(cs);
    if (rc != SSDQ_OK) {
        if (g->exec) cudaGraphExecDestroy(g->exec);
        if (g->graph) cudaGraphDestroy(g->graph);
        delete g;
        return rc;
    }
    *out = g;
    return SSDQ_OK;
}

ssdq_status ssd_decode_graph_launch(ssdq_graph* g, void* stream) {
    if (!g || !g->exec) return fail(SSDQ_ERR_NULL, "graph handle is NULL");
    const cudaError_t e = cudaGraphLaunch(g->exec, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail(SSDQ_ERR_CUDA, "cudaGraphLaunch: %s", cudaGetErrorString(e));
    g_launches.fetch_add((uint64_t)g->steps * g->n_layers + 1u, std::memory_order_relaxed);
    return SSDQ_OK;
}

ssdq_status ssd_decode_graph_destroy(ssdq_graph* g) {
    if (!g) return SSDQ_OK;
    if (g->exec) cudaGraphExecDestroy(g->exec);
    if (g->graph) cudaGraphDestroy(g->graph);
    delete g;
    return SSDQ_OK;
}

ssdq_status ssdq_copy(const void* src, void* dst, uint64_t bytes, void* stream) {
    if (bytes == 0) return SSDQ_OK;
    if (!src || !dst) return fail(SSDQ_ERR_NULL, "src and dst are required");
    if (bytes % 16 != 0) return fail(SSDQ_ERR_SHAPE, "bytes must be a multiple of 16");
    if (!aligned16(src) || !aligned16(dst)) return fail(SSDQ_ERR_ALIGN, "src and dst must be 16-byte aligned");
    return cuda_result(ssdq::launch_copy(src, dst, bytes, static_cast<cudaStream_t>(stream)), "copy kernel");
}

ssdq_status ssdq_debug_status(uint32_t* out4, int reset) {
#ifdef SSDQ_DEBUG
    if (!out4) return fail(SSDQ_ERR_NULL, "out4 is NULL");
    uint32_t* dev = debug_status_address();
    if (!dev) return fail(SSDQ_ERR_CUDA, "no address for the debug status words");
    cudaError_t e = cudaMemcpy(out4, dev, 4 * sizeof(uint32_t), cudaMemcpyDeviceToHost);      // synchronises with earlier work
    if (e == cudaSuccess && reset) e = cudaMemset(dev, 0, 4 * sizeof(uint32_t));
    if (e != cudaSuccess) return fail(SSDQ_ERR_CUDA, "debug status: %s", cudaGetErrorString(e));
    return SSDQ_OK;
#else
    (void)out4; (void)reset;
    return fail(SSDQ_ERR_UNSUPPORTED, "not a bounds-checking build (compile with -DSSDQ_DEBUG)");
#endif
}

const char* ssdq_last_kernel(void) {
    switch (g_last_kernel) {
        case 0: return "ssd_update_kernel";
        case 1: return "ssd_update_tile_kernel";
        case 2: return "ssd_update_stream_kernel";
        case 3: return "ssd_update_headscale_kernel";
        case 4: return "ssd_update_mamba1_kernel";
        default: return "";
    }
}

const char* ssdq_last_error(void) { return g_err; }

int ssdq_set_launch_overlap(int enabled) { return g_launch_overlap.exchange(enabled != 0, std::memory_order_relaxed); }

uint64_t ssdq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"

// ssdq_metrics.cu -- sanity metrics of a quantised trajectory against its full-precision twin:
// the state error sum (h_hat - h)^2 / sum h^2 of the open-loop replay (Appendix B "Open-loop replay"),
// kept per head so that it can be binned by memory length, and a KL divergence between softmax
// distributions over the readout vector of each sequence (a surrogate of Section 4's per-token KL: there is
// no vocabulary here).
#include <mutex>

#include "../../include/ssdq.h"
#include "ssdq_update.cuh"

namespace ssdq {

constexpr int kMetricThreads = 256;

__device__ __forceinline__ double block_sum(double v, double* smem) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    __syncthreads();
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < kMetricThreads / 32; ++w) t += smem[w];     // same order on every thread
    return t;
}

// Pass 1: one CTA per (b, h) item; partial[item] = (sum (h_hat - h)^2, sum h^2) over the item's P*N entries.
template <int FMT>
__global__ void __launch_bounds__(kMetricThreads) state_error_partial_kernel(const uint4* __restrict__ codes,
                                                                             const float* __restrict__ scales,
                                                                             const float* __restrict__ twin,
                                                                             uint32_t item_elems, uint32_t scale_block,
                                                                             double2* __restrict__ partial) {
    constexpr int EPL = Fmt<FMT>::kEpl;
    __shared__ double smem[kMetricThreads / 32];
    const uint64_t item = blockIdx.x;
    const uint64_t first = item * item_elems;
    double e2 = 0.0, r2 = 0.0;
    for (uint32_t i = threadIdx.x * EPL; i < item_elems; i += kMetricThreads * EPL) {
        float h[EPL];
        unpack_lane<FMT>(codes[(first + i) / EPL], h);
        if constexpr (Fmt<FMT>::kScaled) {
            const float s = scales[(first + i) / scale_block];
#pragma unroll
            for (int j = 0; j < EPL; ++j) h[j] = __fmul_rn(h[j], s);
        }
#pragma unroll
        for (int j = 0; j < EPL; ++j) {
            const double ref = (double)twin[first + i + j];
            const double d = (double)h[j] - ref;
            e2 += d * d;
            r2 += ref * ref;
        }
    }
    e2 = block_sum(e2, smem);
    r2 = block_sum(r2, smem);
    if (threadIdx.x == 0) partial[item] = make_double2(e2, r2);
}

// Pass 2: one thread per head sums its items over the batch in a fixed order (run-to-run identical).
__global__ void state_error_finish_kernel(const double2* __restrict__ partial, uint32_t batch, uint32_t nheads,
                                          double* __restrict__ err2, double* __restrict__ ref2) {
    const uint32_t h = blockIdx.x * blockDim.x + threadIdx.x;
    if (h >= nheads) return;
    double e = 0.0, r = 0.0;
    for (uint32_t b = 0; b < batch; ++b) {
        const double2 p = partial[(uint64_t)b * nheads + h];
        e += p.x;
        r += p.y;
    }
    err2[h] = e;
    ref2[h] = r;
}

cudaError_t launch_state_error(const void* codes, const float* scales, const float* twin, uint32_t batch, uint32_t nheads,
                               uint32_t item_elems, int fmt, uint32_t scale_block, double* err2, double* ref2,
                               void* workspace, cudaStream_t s) {
    const uint32_t n_items = batch * nheads;
    double2* partial = reinterpret_cast<double2*>(workspace);
    const uint4* c = reinterpret_cast<const uint4*>(codes);
    switch (fmt) {
        case FMT_FP16: state_error_partial_kernel<FMT_FP16><<<n_items, kMetricThreads, 0, s>>>(c, scales, twin, item_elems, scale_block, partial); break;
        case FMT_BF16: state_error_partial_kernel<FMT_BF16><<<n_items, kMetricThreads, 0, s>>>(c, scales, twin, item_elems, scale_block, partial); break;
        case FMT_E4M3: state_error_partial_kernel<FMT_E4M3><<<n_items, kMetricThreads, 0, s>>>(c, scales, twin, item_elems, scale_block, partial); break;
        case FMT_INT: state_error_partial_kernel<FMT_INT><<<n_items, kMetricThreads, 0, s>>>(c, scales, twin, item_elems, scale_block, partial); break;
        case FMT_FP32: state_error_partial_kernel<FMT_FP32><<<n_items, kMetricThreads, 0, s>>>(c, scales, twin, item_elems, scale_block, partial); break;
        default: return cudaErrorInvalidValue;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    state_error_finish_kernel<<<(nheads + 127) / 128, 128, 0, s>>>(partial, batch, nheads, err2, ref2);
    return cudaGetLastError();
}

// KL(p || q) with p = softmax(y_ref[b, :]), q = softmax(y_q[b, :]); one CTA per sequence.
__global__ void __launch_bounds__(kMetricThreads) readout_kl_kernel(const float* __restrict__ y_ref, const float* __restrict__ y_q,
                                                                    uint32_t width, float* __restrict__ kl) {
    __shared__ double smem[kMetricThreads / 32];
    __shared__ float fmax_s[2][kMetricThreads / 32];
    const float* a = y_ref + (uint64_t)blockIdx.x * width;
    const float* b = y_q + (uint64_t)blockIdx.x * width;
    float ma = -INFINITY, mb = -INFINITY;
    for (uint32_t i = threadIdx.x; i < width; i += kMetricThreads) { ma = fmaxf(ma, a[i]); mb = fmaxf(mb, b[i]); }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        ma = fmaxf(ma, __shfl_xor_sync(0xFFFFFFFFu, ma, off));
        mb = fmaxf(mb, __shfl_xor_sync(0xFFFFFFFFu, mb, off));
    }
    if (threadIdx.x % 32 == 0) { fmax_s[0][threadIdx.x / 32] = ma; fmax_s[1][threadIdx.x / 32] = mb; }
    __syncthreads();
    for (int w = 0; w < kMetricThreads / 32; ++w) { ma = fmaxf(ma, fmax_s[0][w]); mb = fmaxf(mb, fmax_s[1][w]); }
    // log-sum-exp of both rows, then sum p (log p - log q)
    double sa = 0.0, sb = 0.0;
    for (uint32_t i = threadIdx.x; i < width; i += kMetricThreads) { sa += exp((double)a[i] - ma); sb += exp((double)b[i] - mb); }
    sa = block_sum(sa, smem);
    sb = block_sum(sb, smem);
    const double lza = (double)ma + log(sa), lzb = (double)mb + log(sb);
    double acc = 0.0;
    for (uint32_t i = threadIdx.x; i < width; i += kMetricThreads) {
        const double lp = (double)a[i] - lza, lq = (double)b[i] - lzb;
        acc += exp(lp) * (lp - lq);
    }
    acc = block_sum(acc, smem);
    if (threadIdx.x == 0) kl[blockIdx.x] = (float)acc;
}

// Plain 128-bit copy, grid-stride: the floor that a state update is timed against (Table 11, "copy").  Two independent
// loads in flight per thread and 16 CTAs of 512 threads per SM was the fastest of a sweep on this part.
__global__ void __launch_bounds__(512) copy_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, uint64_t n_vec) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + stride < n_vec; i += 2 * stride) {
        const uint4 a = src[i], b = src[i + stride];
        dst[i] = a;
        dst[i + stride] = b;
    }
    if (i < n_vec) dst[i] = src[i];
}
cudaError_t launch_copy(const void* src, void* dst, uint64_t bytes, cudaStream_t s) {
    const uint64_t n_vec = bytes / 16;
    uint64_t grid = (n_vec + 511) / 512;
    if (grid > 148u * 16u) grid = 148u * 16u;
    copy_kernel<<<(unsigned)grid, 512, 0, s>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst), n_vec);
    return cudaGetLastError();
}

__global__ void counter_add_kernel(uint32_t* counter, uint32_t n) { *counter += n; }
cudaError_t launch_counter_add(uint32_t* counter, uint32_t n, cudaStream_t s) {
    counter_add_kernel<<<1, 1, 0, s>>>(counter, n);
    return cudaGetLastError();
}

cudaError_t launch_readout_kl(const float* y_ref, const float* y_q, uint32_t batch, uint32_t width, float* kl, cudaStream_t s) {
    readout_kl_kernel<<<batch, kMetricThreads, 0, s>>>(y_ref, y_q, width, kl);
    return cudaGetLastError();
}

}  // namespace ssdq

// ---------------------------------------------------------------------------------------------
// ssdq_state_error_static: the state-error metric for callers that cannot hand over a workspace.
// Its scratch (the per-(b, h) partial sums between the two passes) lives in this fixed device array,
// which every GPU that loads the library carries until the process exits.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr uint32_t kStaticMaxItems = SSDQ_STATE_ERROR_STATIC_MAX_ITEMS;          // (b, h) pairs
static __device__ __align__(256) double2 g_static_partials[kStaticMaxItems];    // 1 MiB

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
double2* g_static_ptr[kMaxDevices] = {};     // device address of g_static_partials, per device ordinal

// In host code the name g_static_partials is only a stand-in for the symbol, not a device address: the
// address valid on the current device has to be asked for.  Done once per device, on the first call there.
ssdq_status static_scratch_for_current_device(double2** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (ssdq_status)ssdq::report_failure(SSDQ_ERR_CUDA, cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return (ssdq_status)ssdq::report_failure(SSDQ_ERR_UNSUPPORTED, "device ordinal beyond the static table");
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_partials);
        if (e != cudaSuccess || !ptr) return (ssdq_status)ssdq::report_failure(SSDQ_ERR_CUDA, e != cudaSuccess ? cudaGetErrorString(e) : "no address for the static scratch");
        g_static_ptr[dev] = static_cast<double2*>(ptr);
    }
    *out = g_static_ptr[dev];
    return SSDQ_OK;
}

}  // namespace

extern "C" ssdq_status ssdq_state_error_static(const void* codes, const float* scales, const float* twin, uint32_t batch,
                                       uint32_t nheads, uint32_t headdim, uint32_t dstate, int format,
                                       uint32_t scale_block, double* err2_per_head, double* ref2_per_head, void* stream) {
    if (format < SSDQ_FP16 || format > SSDQ_INT4) return (ssdq_status)ssdq::report_failure(SSDQ_ERR_UNSUPPORTED, "unknown format");
    if (batch == 0 || nheads == 0 || headdim == 0 || dstate == 0) return (ssdq_status)ssdq::report_failure(SSDQ_ERR_SHAPE, "sizes must be positive");
    if (((uint64_t)headdim * dstate) % 16 != 0) return (ssdq_status)ssdq::report_failure(SSDQ_ERR_SHAPE, "headdim * dstate must be a multiple of 16");
    if ((uint64_t)batch * nheads > kStaticMaxItems)
        return (ssdq_status)ssdq::report_failure(SSDQ_ERR_SHAPE, "batch * nheads exceeds SSDQ_STATE_ERROR_STATIC_MAX_ITEMS (65536): "
                                                   "use ssdq_state_error with a caller-owned workspace");
    if (!codes || !twin || !err2_per_head || !ref2_per_head) return (ssdq_status)ssdq::report_failure(SSDQ_ERR_NULL, "codes, twin and outputs are required");
    if ((reinterpret_cast<uintptr_t>(codes) & 15u) || (reinterpret_cast<uintptr_t>(twin) & 3u))
        return (ssdq_status)ssdq::report_failure(SSDQ_ERR_ALIGN, "codes must be 16-byte aligned");
    const bool scaled = format == SSDQ_E4M3 || format >= SSDQ_INT8;
    if (scaled && (!scales || scale_block == 0 || scale_block % 16 != 0))
        return (ssdq_status)ssdq::report_failure(SSDQ_ERR_SHAPE, "scaled stores need scales and a scale_block that is a multiple of 16");
    double2* scratch = nullptr;
    const ssdq_status rc = static_scratch_for_current_device(&scratch);
    if (rc != SSDQ_OK) return rc;
    // every partial the second pass reads is written by the first pass of this same call: nothing has to be cleared
    const cudaError_t e = ssdq::launch_state_error(codes, scales, twin, batch, nheads, headdim * dstate,
                                                   format >= SSDQ_INT8 ? (int)ssdq::FMT_INT : format, scale_block,
                                                   err2_per_head, ref2_per_head, scratch, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return (ssdq_status)ssdq::report_failure(SSDQ_ERR_CUDA, cudaGetErrorString(e));
    ssdq::count_launches(2);
    return SSDQ_OK;
}

// ssdq_internal.h -- host/device plain-data structures passed between the C ABI and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "ssdq_device.cuh"

namespace ssdq {

// Debug builds (-DSSDQ_DEBUG) carry the extents of the caller's buffers into every update kernel: each lane checks the
// index ranges it derives against them before it touches memory, records the first violation in a status word and skips
// its accesses (no trap), and the C ABI reports the word (ssdq_debug_status).  Release builds compile none of this.
#ifdef SSDQ_DEBUG
struct DebugBounds {
    uint32_t* status;        // [4] device words: code, index low, index high, blockIdx.x of the first violation
    uint64_t state_vecs;     // 16-byte vectors in the state
    uint64_t rows;           // B * H * P: extent of x, y (and z)
    uint64_t scales;         // FP32 scales
    uint64_t items;          // B * H: extent of dt
    uint64_t bc_floats;      // B * G * N: extent of Bm, Cm
};
#endif

// Kernel parameters of one fused update launch (copied by value into constant memory at launch).
struct UpdateParams {
    void* state;
    float* scales;
    const float* x;
    const float* dt;
    const float* A;
    const float* Bm;
    const float* Cm;
    const float* D;
    const float* dt_bias;    // [H] or null
    const float* z;          // [B,H,P] or null: y <- y * silu(z)
    float* y;
    uint32_t B, H, P, N;
    uint32_t dt_softplus;    // dt <- softplus_spec(dt + dt_bias)
    uint32_t ngroups;        // B, C are [B, G, N]
    uint32_t heads_per_group;
    uint32_t n_items;        // B * H
    uint32_t scale_block;    // scaled stores: 16 or N
    float scale_top;         // scaled stores: block scale = amax / scale_top (448 for E4M3, q_max for INTb)
    float inv_scale_top;     // RN(1 / scale_top)
    uint32_t step_t;
    const uint32_t* step_base;   // null, or a device word added to step_t (replayable graphs keep their step count there)
    uint32_t layer;
    // global row of local row (b, h, p) = local row + row_off0 + b * row_skip  (rows of the [B_global * H_global * P, N] view):
    uint64_t row_off0;       // (batch_index_base * H_global + head_index_base) * P
    uint32_t row_skip;       // (H_global - H) * P: rows of other head shards between two local sequences
    uint32_t spi;            // slots per (b, h) item inside a CTA (power of two)
    uint32_t items_per_cta;
    uint32_t rps;            // rows per slot
    WeylConst weyl;
    uint64_t sr_seed;
    uint32_t overlap;        // 0: plain launch; else programmatic stream serialization: 1 wait, then release the successor; 2 release first
    uint32_t prepare_only;   // host side only: pick the kernel and do its one-time set-up (attributes, occupancy), launch nothing
#ifdef SSDQ_DEBUG
    DebugBounds dbg;
#endif
};

// Parameters of quantize_store / replay / dequantize / thresholds.
struct QuantParams {
    const float* src;
    const float* decay;       // replay only: one decay per rows_per_decay consecutive rows
    uint32_t rows_per_decay;
    void* codes;
    float* scales;
    uint64_t n_rows;
    uint32_t row_len;
    uint32_t scale_block;
    float scale_top;
    uint32_t step_t;
    uint32_t layer;
    uint64_t row_base;
    uint64_t rows_per_seq;    // 0, or rows of one local sequence: global row = row_base + row + (row / rows_per_seq) * row_skip
    uint32_t row_skip;
    WeylConst weyl;
    uint64_t sr_seed;
};

// one translation unit per storage format
cudaError_t launch_update_fp16(const UpdateParams& p, int rule, bool a_per_state, cudaStream_t s);
cudaError_t launch_update_bf16(const UpdateParams& p, int rule, bool a_per_state, cudaStream_t s);
cudaError_t launch_update_e4m3(const UpdateParams& p, int rule, bool a_per_state, cudaStream_t s);
cudaError_t launch_update_fp32(const UpdateParams& p, int rule, bool a_per_state, cudaStream_t s);
cudaError_t launch_update_int8(const UpdateParams& p, int rule, bool a_per_state, cudaStream_t s);

cudaError_t launch_quantize(const QuantParams& p, int fmt, int rule, cudaStream_t s);   // p.decay != null: replay step
cudaError_t launch_dequantize(const void* codes, const float* scales, uint64_t n, int fmt, uint32_t scale_block,
                              float* out, cudaStream_t s);
cudaError_t launch_thresholds(int rule, const WeylConst& w, uint64_t sr_seed, uint32_t layer, uint64_t first_flat,
                              uint64_t n, uint32_t step_t, uint32_t* out, cudaStream_t s);

cudaError_t launch_state_error(const void* codes, const float* scales, const float* twin, uint32_t batch, uint32_t nheads,
                               uint32_t item_elems, int fmt, uint32_t scale_block, double* err2, double* ref2,
                               void* workspace, cudaStream_t s);
// error text / launch counter of the C ABI, for entry points defined outside ssdq_api.cu
int report_failure(int status, const char* text);
void note_kernel(int family);      // 0 generic, 1 tile, 2 stream: which fused-update kernel the launcher picked
void count_launches(unsigned n);

cudaError_t launch_copy(const void* src, void* dst, uint64_t bytes, cudaStream_t s);
cudaError_t launch_counter_add(uint32_t* counter, uint32_t n, cudaStream_t s);
cudaError_t launch_readout_kl(const float* y_ref, const float* y_q, uint32_t batch, uint32_t width, float* kl, cudaStream_t s);

}  // namespace ssdq

/* ssdq.h -- C ABI of the quantized selective-state-update decode library (CUDA, sm_100a).
 *
 * The library keeps a Mamba-style recurrent state in a low-precision store -- FP16, BF16, FP8-E4M3
 * with an FP32 block scale, or symmetric block-absmax integers INT8/7/6/4 with an FP32 block scale
 * (Appendix B "Formats"); FP32 is the unrounded twin -- and, once per generated token and layer,
 * makes one fused pass over it: dequantise, h' = exp(dt*A)*h + dt*B*x (Eq. 1; Appendix B "Runners"),
 * read out y = C.h' + D*x from the unrounded h', and write h' back rounded by Eq. 2 under one of four
 * threshold rules (Section 2 "Rounding with a threshold"): round-to-nearest, stochastic rounding
 * driven by counter-based Philox4x32-10 or by a cheap integer hash (Section 6.5 "Cost"), or the
 * golden-ratio Weyl dither in its 32-bit integer form (Appendix B "Dithers").
 *
 * Conventions for every entry point
 *   - Pointers named in a descriptor are DEVICE pointers unless stated; descriptors themselves are
 *     HOST memory and are copied by value at launch.  The caller owns all memory.  Unless an entry
 *     point says otherwise the library allocates nothing on the device.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls enqueue
 *     work and return; they do not synchronise.
 *   - Every argument check happens before any launch; a failed check launches nothing.
 *   - Return value: SSDQ_OK or a negative ssdq_status; ssdq_last_error() gives a thread-local text.
 *   - Indices that feed the thresholds are GLOBAL: entry (b, h, p, n) of a layer has flat index
 *     ((( b + batch_index_base) * H_global + h + head_index_base) * P + p) * N + n, with H_global =
 *     nheads_global (or H when that field is 0), so a shard of the batch, of the heads, or of both
 *     reproduces the bits of the unsharded run.  All tensors of a call hold the shard only.
 *   - All inputs must be finite.  Binary32 subnormals are honoured (no flush to zero).
 */
#ifndef SSDQ_H_
#define SSDQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SSDQ_OK = 0,
    SSDQ_ERR_NULL = -1,         /* a required pointer is NULL */
    SSDQ_ERR_SHAPE = -2,        /* a size is zero or inconsistent */
    SSDQ_ERR_ALIGN = -3,        /* a pointer is not aligned as documented */
    SSDQ_ERR_UNSUPPORTED = -4,  /* a valid request this build has no kernel for */
    SSDQ_ERR_CUDA = -5          /* the CUDA runtime reported an error (see ssdq_last_error) */
} ssdq_status;

/* Storage formats (Appendix B "Formats").  SSDQ_FP32 stores binary32 and never rounds: it is the
 * full-precision twin that the quantised trajectory is compared with. */
typedef enum {
    SSDQ_FP16 = 0, SSDQ_BF16 = 1, SSDQ_E4M3 = 2, SSDQ_FP32 = 3,
    /* Symmetric block-absmax integers (Appendix B "Formats", INTb): one int8 per entry holding k in
     * [-q_max, q_max], q_max = 2^(b-1) - 1 = 127 / 63 / 31 / 7, value = k * s with the FP32 block scale
     * s = max(amax_block / q_max, FLT_MIN).  The grid is uniform, so Eq. 2 is floor(v + u) on v = h' * (1/s). */
    SSDQ_INT8 = 4, SSDQ_INT7 = 5, SSDQ_INT6 = 6, SSDQ_INT4 = 7
} ssdq_format;

/* Threshold rules of Eq. 2.  RTN rounds to nearest, ties to even (the rule of native casts).
 * SSDQ_SR_HASH is stochastic rounding driven by a cheap integer hash instead of Philox (Section 6.5 "Cost";
 * Appendix B "Decode regime"): U = fmix32(i_lo*0x9E3779B1 + t*0x85EBCA77 + layer*0xC2B2AE3D + seed_lo*0x27D4EB2F
 * + (i_hi ^ seed_hi)*0x165667B1) >> 8 with i the flat entry index, seed = sr_seed, fmix32 the MurmurHash3 finaliser. */
typedef enum { SSDQ_RTN = 0, SSDQ_SR_PHILOX = 1, SSDQ_WEYL = 2, SSDQ_SR_HASH = 3 } ssdq_rule;

/* Weyl dither in 32-bit fixed point (Appendix B "Dithers", hardware form):
 *   acc(r, c, t) = mul_row*(r+1) + mul_col*(c+1) + base + t*phi   (mod 2^32),   u = (acc >> 8) / 2^24
 * with r = flat / block and c = flat % block.  Plain data, 32 bytes, no pointers. */
typedef struct {
    uint32_t mul_row;   /* 0.7548776662 * 2^32 */
    uint32_t mul_col;   /* 0.5698402910 * 2^32 */
    uint32_t phi;       /* 2654435769, the golden-ratio increment */
    uint32_t base;      /* 0.1234567*2^32 * layer + 0.3141592*2^32 * seed  (mod 2^32) */
    uint32_t block;     /* entries per dither block along the state dimension: 16, or N */
    uint32_t layer;
    uint32_t seed;
    uint32_t reserved;
} ssdq_weyl;

/* Fill `out` (HOST) for layer `layer` and offset seed `seed` (the paper's sigma; 0 in its runs).
 * `block` must be a positive multiple of 16.  Pure host arithmetic; no CUDA call. */
ssdq_status weyl_offsets_init(ssdq_weyl* out, uint32_t layer, uint32_t seed, uint32_t block);

/* Test aid: write the 24-bit thresholds U of entries flat = first_flat .. first_flat + n - 1 at
 * write index step_t into out_u24 (DEVICE, n x uint32).  rule = SSDQ_WEYL uses `weyl`;
 * SSDQ_SR_PHILOX uses Philox4x32-10 with key = sr_seed and counter = (flat/4 low, flat/4 high,
 * step_t, layer), word flat % 4, top 24 bits; SSDQ_SR_HASH as defined at ssdq_rule; SSDQ_RTN writes zeros. */
ssdq_status ssdq_thresholds_materialize(int rule, const ssdq_weyl* weyl, uint64_t sr_seed, uint32_t layer,
                                uint64_t first_flat, uint64_t n, uint32_t step_t, uint32_t* out_u24, void* stream);

/* One layer's decode-step problem. */
typedef struct {
    uint32_t batch, nheads, headdim, dstate;  /* B, H, P, N.  N in {16, 32, 64, 128, 256} (E4M3: N >= 16;
                                                 FP32: N >= 16).  Mamba-1 is H = d_inner, P = 1. */
    void* state;         /* [B, H, P, N] codes of `format`, N contiguous, 16-byte aligned; updated IN PLACE */
    float* scales;       /* E4M3 and INTb: [B, H, P, N / scale_block] FP32 block scales, updated in place */
    uint32_t scale_block;/* E4M3 and INTb: 16 or N (entries along N that share one scale) */
    int32_t format;      /* ssdq_format */
    const float* x;      /* [B, H, P] */
    const float* dt;     /* [B, H], already passed through softplus */
    const float* A;      /* [H] (one decay per head) or [H, N] if a_per_state; [H, N] must be 16-byte aligned */
    const float* Bm;     /* [B, N], one group, 16-byte aligned */
    const float* Cm;     /* [B, N], one group, 16-byte aligned */
    const float* D;      /* [H] or NULL (no skip term) */
    uint32_t a_per_state;/* 0: A is [H]; 1: A is [H, N] (Mamba-1) */
    float* y;            /* [B, H, P] output */
    int32_t rule;        /* ssdq_rule */
    ssdq_weyl weyl;      /* used when rule == SSDQ_WEYL; weyl.block must be 16 or N */
    uint64_t sr_seed;    /* Philox key when rule == SSDQ_SR_PHILOX */
    uint32_t layer;      /* layer index in the SR counter (the Weyl layer term sits in weyl.base) */
    uint32_t batch_index_base;  /* global index of local sequence 0 */
    /* The rest of a production selective-state-update signature (Appendix B "Runners" keeps the grouped B and C and
     * the output gate of the Mamba implementations it follows).  All optional: zero / NULL gives the plain step. */
    const float* dt_bias;/* [H] or NULL: added to dt (one rounded add) */
    const float* z;      /* [B, H, P] or NULL: y <- y * z * sigmoid(z) */
    uint32_t dt_softplus;/* 1: dt <- softplus_spec(dt + dt_bias), the library's fixed binary32 softplus */
    uint32_t ngroups;    /* G > 1: Bm, Cm are [B, G, N] and head h reads group h / (H / G); 0 or 1: one group.
                            Heads and groups are those of this call's tensors (a head shard carries its own groups). */
    /* Head shard (tensor parallel): this call holds heads head_index_base .. head_index_base + H - 1 of a layer with
     * nheads_global heads.  Only the threshold indices change.  0, 0 = the call holds every head. */
    uint32_t head_index_base;   /* global index of local head 0 */
    uint32_t nheads_global;     /* 0 = nheads; otherwise >= head_index_base + nheads */
} ssdq_update_desc;

/* One fused decode step of one layer (Eq. 1, readout, Eq. 2), in place, one kernel launch:
 *   h  = dequant(state)                          (E4M3: code * scale, one rounded multiply)
 *   dt = softplus_spec(dt + dt_bias) if dt_softplus (else dt + dt_bias, else dt)
 *   a  = exp_spec(dt*A);  w = (dt*x)*B;  h' = fma(a, h, w)      all binary32, in this order
 *   y  = (sum_n C[n]*h'[n] + D*x) [* z*sigmoid(z)]   (FP32 accumulation, tree order unspecified)
 *   E4M3 / INTb: s = max(amax_block(h') / top, FLT_MIN) with top = 448 / q_max, v = h' * (1/s);  otherwise v = h'
 *   state = encode(Q_u(v)) with u from `rule` at write index step_t (first write is step_t = 1)
 * exp_spec is the library's fixed binary32 exponential (clamp to [-87, 88], Cody-Waite reduction,
 * degree-7 polynomial), identical bit for bit on every call.  Values beyond the format's largest
 * finite number saturate to it; a value rounded to zero keeps its sign. */
ssdq_status ssd_state_update(const ssdq_update_desc* d, uint32_t step_t, void* stream);

/* Quantise an FP32 array into a store with the same rounding functions (Eq. 2): used to seed h_0
 * from a full-precision state (the paper quantises the end-of-prefill state) and to exercise the
 * rules in isolation.  src [n_rows, row_len] DEVICE floats (16-byte aligned); dst_codes
 * [n_rows, row_len] codes (16-byte aligned); dst_scales [n_rows, row_len / scale_block] for E4M3
 * else NULL.  row_len obeys the same limits as dstate; entry (row, col) has flat index
 * (row_index_base + row) * row_len + col. */
ssdq_status quantize_store(const float* src, void* dst_codes, float* dst_scales, uint64_t n_rows, uint32_t row_len,
                   uint32_t scale_block, int format, int rule, const ssdq_weyl* weyl, uint64_t sr_seed,
                   uint32_t layer, uint64_t row_index_base, uint32_t step_t, void* stream);

/* Open-loop replay of recorded traces (Appendix B "Open-loop replay"): h_t = Q(a_t h_{t-1} + w_t), in place on a
 * store.  w [n_rows, row_len] DEVICE floats (16-byte aligned) are the recorded writes, decay [n_rows / rows_per_decay]
 * the recorded decays (rows_per_decay consecutive rows -- a head of P rows -- share one); codes / scales, the rule,
 * its indices and step_t are those of quantize_store.  h' = fma(a, dequant(code), w) in binary32, then block scale,
 * threshold and Eq. 2 exactly as in ssd_state_update (whose state it reproduces bit for bit when fed a = exp_spec(dt*A)
 * and w = (dt*x)*B). */
ssdq_status ssd_replay_step(const float* w, const float* decay, uint32_t rows_per_decay, void* codes, float* scales, uint64_t n_rows,
                    uint32_t row_len, uint32_t scale_block, int format, int rule, const ssdq_weyl* weyl, uint64_t sr_seed,
                    uint32_t layer, uint64_t row_index_base, uint32_t step_t, void* stream);

/* Inverse view of a store: out[i] = decode(code[i]) (* scale[i / scale_block] for E4M3), DEVICE. */
ssdq_status ssdq_dequantize(const void* codes, const float* scales, uint64_t n, int format, uint32_t scale_block,
                    float* out, void* stream);

/* Per-step inputs of the multi-step driver: element (t, l) of tensor X starts at
 * X + (((t - t_first) % ring) * n_layers + l) * stride_X floats, all DEVICE memory. */
typedef struct {
    const float* x;   uint64_t stride_x;    /* each [B, H, P] */
    const float* dt;  uint64_t stride_dt;   /* each [B, H] */
    const float* Bm;  uint64_t stride_B;    /* each [B, N] */
    const float* Cm;  uint64_t stride_C;    /* each [B, N] */
    float* y;         uint64_t stride_y;    /* each [B, H, P]; written for every (t, l) slot of the ring */
    uint32_t ring;    /* number of distinct steps stored (>= 1; == n_steps when every step has its own inputs) */
    uint32_t reserved;
    const float* z;   uint64_t stride_z;    /* each [B, H, P], or NULL: no gate */
} ssdq_step_inputs;

/* T-step decode driver (the open-loop replay of Appendix B run forward): for t = t_first ..
 * t_first + n_steps - 1 and l = 0 .. n_layers - 1, one ssd_state_update launch of layers[l] with
 * write index t and the inputs of slot (t, l), all on `stream`, no host synchronisation.  The
 * x / dt / Bm / Cm / y / z members of layers[l] are ignored (taken from `in`). */
ssdq_status ssd_decode_run(const ssdq_update_desc* layers, uint32_t n_layers, uint32_t t_first, uint32_t n_steps,
                   const ssdq_step_inputs* in, void* stream);

/* Replayable CUDA graph of the decode loop, for decode at small batch where the per-layer launches are bound by launch
 * latency.  ssd_decode_graph_create captures `steps_per_launch` decode steps (steps_per_launch * n_layers fused update
 * launches, inputs of step i from ring slot i % in->ring; steps_per_launch must be a multiple of in->ring) into a graph
 * whose kernels read their write index from DEVICE memory: step i of a launch writes with index *step_counter + 1 + i, and
 * a last node adds steps_per_launch to *step_counter.  The caller owns the counter word (set it to the number of writes
 * done so far, 0 for a fresh state) and every buffer the descriptors name; all must outlive the graph.
 * ssd_decode_graph_launch enqueues one replay on `stream`; the caller refreshes the input ring between replays.
 * The results equal those of ssd_decode_run for the same write indices.  Creation allocates driver-side graph objects
 * (no device memory of the library's own). */
typedef struct ssdq_graph ssdq_graph;
ssdq_status ssd_decode_graph_create(ssdq_graph** out, const ssdq_update_desc* layers, uint32_t n_layers, uint32_t steps_per_launch,
                            const ssdq_step_inputs* in, uint32_t* step_counter);
ssdq_status ssd_decode_graph_launch(ssdq_graph* graph, void* stream);
ssdq_status ssd_decode_graph_destroy(ssdq_graph* graph);

/* Periodic checkpointing (Section 6.5 "Periodic checkpointing"; Appendix B "Decode regime", CC = 8): the state lives in
 * full precision between checkpoints and only every `every`-th write, counted from t_first, is rounded into the store.
 * work_fp32[l] is a caller-owned DEVICE buffer [B, H, P, N] of floats holding layer l's working state (on entry: the
 * dequantised store, or zeros for h_0 = 0).  Per step and layer: one FP32 update launch; on checkpoint steps also
 * quantize_store (work -> layers[l].state under the layer's rule at write index t) and ssdq_dequantize (store -> work).
 * With every == 1 the stores and y equal those of ssd_decode_run.  dstate <= 128. */
ssdq_status ssd_decode_run_checkpointed(const ssdq_update_desc* layers, float* const* work_fp32, uint32_t n_layers, uint32_t every,
                                uint32_t t_first, uint32_t n_steps, const ssdq_step_inputs* in, void* stream);

/* The same driver for callers whose per-step inputs and outputs live in HOST memory (the usual case when the
 * rest of the model runs elsewhere): `host` describes HOST arrays (page-locked memory for full speed) laid out like
 * ssdq_step_inputs, the inputs of step t at ring slot (t - t_first) % host->ring and its y written to the same
 * slot; `staging` describes caller-owned DEVICE buffers with 2 to 8 ring slots and the same strides as `host`.
 * Per step: the inputs of all layers go host -> staging on an internal copy stream, the fused updates run on
 * `stream`, y goes staging -> host on a second internal copy stream; events chain the three so that copy-in of step
 * t+1, compute of step t and copy-out of step t-1 overlap.  When all work enqueued on `stream` has completed,
 * every y has reached the host.  The state never leaves the device.  The two streams and the events are created
 * on the first call on a device (host-side driver resources, no device memory).  One call at a time per device. */
ssdq_status ssd_decode_run_host(const ssdq_update_desc* layers, uint32_t n_layers, uint32_t t_first, uint32_t n_steps,
                        const ssdq_step_inputs* host, const ssdq_step_inputs* staging, void* stream);

/* Sanity metric of a quantised trajectory against its full-precision twin (Appendix B "Open-loop replay":
 * state error = sum (h_hat - h)^2 / sum h^2): err2_per_head[h] = sum over b, p, n of (dequant(codes) - twin)^2 and
 * ref2_per_head[h] = sum of twin^2, both DEVICE doubles [nheads], kept per head so that the caller can bin heads
 * by memory length.  codes/scales as in ssdq_update_desc; twin [B, H, P, N] DEVICE floats.  headdim * dstate must
 * be a multiple of 16.  `workspace` is DEVICE scratch of at least ssdq_state_error_workspace_bytes(batch, nheads)
 * bytes, 16-byte aligned, owned by the caller; it holds per-(b, h) partial sums between the two passes (the sums
 * over the batch are taken in a fixed order, so results are identical from run to run). */
uint64_t ssdq_state_error_workspace_bytes(uint32_t batch, uint32_t nheads);
ssdq_status ssdq_state_error(const void* codes, const float* scales, const float* twin, uint32_t batch, uint32_t nheads,
                     uint32_t headdim, uint32_t dstate, int format, uint32_t scale_block, double* err2_per_head,
                     double* ref2_per_head, void* workspace, uint64_t workspace_bytes, void* stream);

/* The same metric for callers that must not allocate.  (No counterpart in the paper: this entry point exists
 * for the way the library is deployed.)  Some callers of a decode library cannot obtain device memory at the
 * moment they want this number: a serving process that gave the whole HBM to its state/KV pool at start-up has
 * nothing left for cudaMalloc to hand out, and a monitoring hook that runs between decode steps cannot afford
 * cudaMalloc/cudaFree there, because both synchronise the device and would stall the decode loop.  This variant
 * therefore takes no workspace and calls no allocating routine: its scratch (16 bytes per (b, h) pair) is a fixed
 * array inside the library's device image, SSDQ_STATE_ERROR_STATIC_MAX_ITEMS pairs = 1 MiB, which every GPU that
 * loads the library holds until the process exits.
 *   - batch * nheads beyond SSDQ_STATE_ERROR_STATIC_MAX_ITEMS is rejected with SSDQ_ERR_SHAPE (use ssdq_state_error).
 *   - The first call on each device looks up the array's address on that device (the device must be current);
 *     make that first call before any stream capture begins.  The address is kept for the life of the process:
 *     it does not survive a cudaDeviceReset of that device.
 *   - All calls share the one array, which keeps the contents of the last call.  Nothing in it has to start at zero
 *     (each call overwrites every slot it later reads), but two calls that overlap on the GPU -- different streams,
 *     or different host threads on the same device -- race on it: serialise them.
 * Arguments and results are those of ssdq_state_error, minus the workspace. */
#define SSDQ_STATE_ERROR_STATIC_MAX_ITEMS 65536u
ssdq_status ssdq_state_error_static(const void* codes, const float* scales, const float* twin, uint32_t batch, uint32_t nheads,
                            uint32_t headdim, uint32_t dstate, int format, uint32_t scale_block, double* err2_per_head,
                            double* ref2_per_head, void* stream);

/* Surrogate of the paper's per-token KL (Section 4 "What we measure"; there is no vocabulary here): for each
 * sequence b, KL(p || q) = sum_i p_i log(p_i / q_i) with p = softmax(y_ref[b, :]) and q = softmax(y_q[b, :]) over the
 * `width` readout values of that sequence.  y_ref, y_q [batch, width] and kl_per_sequence [batch] are DEVICE floats. */
ssdq_status ssdq_readout_kl(const float* y_ref, const float* y_q, uint32_t batch, uint32_t width, float* kl_per_sequence,
                    void* stream);

/* The floor of the timing protocol: a plain 128-bit copy of `bytes` bytes (a multiple of 16; both pointers DEVICE,
 * 16-byte aligned, not overlapping) by a kernel of this library, so that a state update can be timed against a copy
 * of the same buffers launched the same way (the "copy" column of Table 11, Section 6.5 "Cost"). */
ssdq_status ssdq_copy(const void* src, void* dst, uint64_t bytes, void* stream);

/* Bounds-checking build.  A library compiled with -DSSDQ_DEBUG (python -m paper_2609_39185_b200.build --debug gives
 * libssdq_debug.so) makes every fused-update kernel compare the index ranges it derives with the extents implied by the
 * descriptor before touching memory; a lane that would step outside records the first violation and skips its accesses
 * (nothing traps, the context stays usable).  This call waits for earlier work on the device and copies the four status
 * words to out4 (HOST): code (0 = no violation; 1 state, 2 x/y rows, 3 scales, 4 dt items, 5 B/C), offending index low and
 * high word, block index; reset != 0 clears them afterwards.  In a release build it returns SSDQ_ERR_UNSUPPORTED.
 * It stands in for a memory checker on systems where none can be run. */
ssdq_status ssdq_debug_status(uint32_t* out4, int reset);

/* Name of the kernel family that the last fused-update launch issued from this thread used:
 * "ssd_update_stream_kernel" (persistent, one-byte block-scaled stores on head-shaped tiles),
 * "ssd_update_tile_kernel" (one CTA per head), "ssd_update_headscale_kernel" (one scale per head),
 * "ssd_update_mamba1_kernel" (dstate 16, headdim 1, one decay per state) or "ssd_update_kernel" (any shape); "" before
 * the first launch.
 * For benchmark records. */
const char* ssdq_last_kernel(void);

/* Text of the last error on this thread ("" if none).  The pointer stays valid until the next call
 * of the library on the same thread. */
const char* ssdq_last_error(void);

/* Launch overlap inside the multi-launch stream drivers (ssd_decode_run, ssd_decode_run_checkpointed): when enabled
 * (the default) every fused-update launch after the first of a call carries the programmatic-stream-serialization attribute, so its CTAs are scheduled while the previous kernel of the driver drains;
 * each kernel waits for the completion of all earlier grids before it touches memory, so results do not change (the
 * paper has no counterpart: this is launch plumbing).  The drivers' inputs must not be written by other work while a
 * driver call is in flight, which the drivers require anyway.  A single ssd_state_update call never uses the attribute.
 * Graphs are captured without it (plain edges replay faster) and ssd_decode_run_host launches without it (it was
 * measured to lose beside the copy streams).  Returns the previous setting.  Process-wide. */
int ssdq_set_launch_overlap(int enabled);

/* Number of kernels the library has launched in this process (a counter for benchmarks). */
uint64_t ssdq_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SSDQ_H_ */

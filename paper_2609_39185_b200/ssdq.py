"""ctypes binding of the C-ABI CUDA library (``include/ssdq.h``): argument marshalling only.

Every function takes torch CUDA tensors (used as raw device pointers), enqueues the library's kernels
on torch's current stream and returns without synchronising.  There is no fallback: if the compiled
library is missing, or a call is rejected, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

FP16, BF16, E4M3, FP32 = 0, 1, 2, 3
INT8, INT7, INT6, INT4 = 4, 5, 6, 7
RTN, SR, WEYL, SR_HASH = 0, 1, 2, 3
OK, ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_UNSUPPORTED, ERR_CUDA = 0, -1, -2, -3, -4, -5

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libssdq.so")

EXPORTS = ("weyl_offsets_init", "ssdq_thresholds_materialize", "ssd_state_update", "quantize_store",
           "ssdq_dequantize", "ssd_decode_run", "ssd_decode_run_host", "ssd_replay_step", "ssd_decode_run_checkpointed",
           "ssd_decode_graph_create", "ssd_decode_graph_launch", "ssd_decode_graph_destroy", "ssdq_state_error_workspace_bytes", "ssdq_state_error",
           "ssdq_state_error_static", "ssdq_readout_kl", "ssdq_copy", "ssdq_debug_status", "ssdq_last_kernel", "ssdq_last_error", "ssdq_launch_count",
           "ssdq_set_launch_overlap")

_u32, _u64, _i32, _vp = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int32, ctypes.c_void_p


class SsdqError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(f"ssdq status {status}: {text}")
        self.status = status


class Weyl(ctypes.Structure):
    _fields_ = [("mul_row", _u32), ("mul_col", _u32), ("phi", _u32), ("base", _u32), ("block", _u32),
                ("layer", _u32), ("seed", _u32), ("reserved", _u32)]


class UpdateDesc(ctypes.Structure):
    _fields_ = [("batch", _u32), ("nheads", _u32), ("headdim", _u32), ("dstate", _u32),
                ("state", _vp), ("scales", _vp), ("scale_block", _u32), ("format", _i32),
                ("x", _vp), ("dt", _vp), ("A", _vp), ("Bm", _vp), ("Cm", _vp), ("D", _vp),
                ("a_per_state", _u32), ("y", _vp), ("rule", _i32), ("weyl", Weyl), ("sr_seed", _u64),
                ("layer", _u32), ("batch_index_base", _u32), ("dt_bias", _vp), ("z", _vp), ("dt_softplus", _u32),
                ("ngroups", _u32), ("head_index_base", _u32), ("nheads_global", _u32)]


class StepInputs(ctypes.Structure):
    _fields_ = [("x", _vp), ("stride_x", _u64), ("dt", _vp), ("stride_dt", _u64), ("Bm", _vp), ("stride_B", _u64),
                ("Cm", _vp), ("stride_C", _u64), ("y", _vp), ("stride_y", _u64), ("ring", _u32), ("reserved", _u32),
                ("z", _vp), ("stride_z", _u64)]


DEBUG_LIB_PATH = os.path.join(_HERE, "libssdq_debug.so")

_lib = None


def lib() -> ctypes.CDLL:
    """Load libssdq.so (built by ``python -m paper_2609_39185_b200.build``); raises if it is missing."""
    global _lib
    if _lib is None:
        _lib = _load(LIB_PATH)
    return _lib


def _load(path) -> ctypes.CDLL:
    if True:
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: build the CUDA extension first "
                              "(python -m paper_2609_39185_b200.build); there is no CPU fallback")
        L = ctypes.CDLL(path)
        L.weyl_offsets_init.restype = ctypes.c_int
        L.weyl_offsets_init.argtypes = [ctypes.POINTER(Weyl), _u32, _u32, _u32]
        L.ssdq_thresholds_materialize.restype = ctypes.c_int
        L.ssdq_thresholds_materialize.argtypes = [ctypes.c_int, ctypes.POINTER(Weyl), _u64, _u32, _u64, _u64, _u32, _vp, _vp]
        L.ssd_state_update.restype = ctypes.c_int
        L.ssd_state_update.argtypes = [ctypes.POINTER(UpdateDesc), _u32, _vp]
        L.quantize_store.restype = ctypes.c_int
        L.quantize_store.argtypes = [_vp, _vp, _vp, _u64, _u32, _u32, ctypes.c_int, ctypes.c_int, ctypes.POINTER(Weyl),
                                     _u64, _u32, _u64, _u32, _vp]
        L.ssdq_dequantize.restype = ctypes.c_int
        L.ssdq_dequantize.argtypes = [_vp, _vp, _u64, ctypes.c_int, _u32, _vp, _vp]
        L.ssd_decode_run.restype = ctypes.c_int
        L.ssd_decode_run.argtypes = [ctypes.POINTER(UpdateDesc), _u32, _u32, _u32, ctypes.POINTER(StepInputs), _vp]
        L.ssd_replay_step.restype = ctypes.c_int
        L.ssd_replay_step.argtypes = [_vp, _vp, _u32, _vp, _vp, _u64, _u32, _u32, ctypes.c_int, ctypes.c_int, ctypes.POINTER(Weyl),
                                      _u64, _u32, _u64, _u32, _vp]
        L.ssd_decode_run_checkpointed.restype = ctypes.c_int
        L.ssd_decode_run_checkpointed.argtypes = [ctypes.POINTER(UpdateDesc), ctypes.POINTER(_vp), _u32, _u32, _u32, _u32,
                                                  ctypes.POINTER(StepInputs), _vp]
        L.ssd_decode_graph_create.restype = ctypes.c_int
        L.ssd_decode_graph_create.argtypes = [ctypes.POINTER(_vp), ctypes.POINTER(UpdateDesc), _u32, _u32, ctypes.POINTER(StepInputs), _vp]
        L.ssd_decode_graph_launch.restype = ctypes.c_int
        L.ssd_decode_graph_launch.argtypes = [_vp, _vp]
        L.ssd_decode_graph_destroy.restype = ctypes.c_int
        L.ssd_decode_graph_destroy.argtypes = [_vp]
        L.ssd_decode_run_host.restype = ctypes.c_int
        L.ssd_decode_run_host.argtypes = [ctypes.POINTER(UpdateDesc), _u32, _u32, _u32, ctypes.POINTER(StepInputs),
                                          ctypes.POINTER(StepInputs), _vp]
        L.ssdq_state_error_workspace_bytes.restype = _u64
        L.ssdq_state_error_workspace_bytes.argtypes = [_u32, _u32]
        L.ssdq_state_error.restype = ctypes.c_int
        L.ssdq_state_error.argtypes = [_vp, _vp, _vp, _u32, _u32, _u32, _u32, ctypes.c_int, _u32, _vp, _vp, _vp, _u64, _vp]
        L.ssdq_state_error_static.restype = ctypes.c_int
        L.ssdq_state_error_static.argtypes = [_vp, _vp, _vp, _u32, _u32, _u32, _u32, ctypes.c_int, _u32, _vp, _vp, _vp]
        L.ssdq_readout_kl.restype = ctypes.c_int
        L.ssdq_readout_kl.argtypes = [_vp, _vp, _u32, _u32, _vp, _vp]
        L.ssdq_copy.restype = ctypes.c_int
        L.ssdq_copy.argtypes = [_vp, _vp, _u64, _vp]
        L.ssdq_last_kernel.restype = ctypes.c_char_p
        L.ssdq_last_kernel.argtypes = []
        L.ssdq_last_error.restype = ctypes.c_char_p
        L.ssdq_last_error.argtypes = []
        L.ssdq_launch_count.restype = _u64
        L.ssdq_launch_count.argtypes = []
        L.ssdq_set_launch_overlap.restype = ctypes.c_int
        L.ssdq_set_launch_overlap.argtypes = [ctypes.c_int]
        L.ssdq_debug_status.restype = ctypes.c_int
        L.ssdq_debug_status.argtypes = [ctypes.POINTER(_u32 * 4), ctypes.c_int]
    return L


class debug_library:
    """Context manager: inside it every call of this module goes to the bounds-checking build of the library
    (libssdq_debug.so, from ``python -m paper_2609_39185_b200.build --debug``); debug_status() reads its status words."""

    def __enter__(self):
        global _lib
        self._saved = _lib
        _lib = _load(DEBUG_LIB_PATH)
        return self

    def __exit__(self, *exc):
        global _lib
        _lib = self._saved
        return False


def debug_status(reset: bool = True):
    """(code, index, block) of the first out-of-range access the bounds-checking build saw, or (0, 0, 0)."""
    out = (_u32 * 4)()
    _check(lib().ssdq_debug_status(ctypes.byref(out), int(reset)))
    return int(out[0]), int(out[1]) | (int(out[2]) << 32), int(out[3])


def _check(status):
    if status != OK:
        raise SsdqError(status, lib().ssdq_last_error().decode())


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream():
    import torch
    return torch.cuda.current_stream().cuda_stream


def weyl_offsets_init(layer: int = 0, seed: int = 0, block: int = 16) -> Weyl:
    w = Weyl()
    _check(lib().weyl_offsets_init(ctypes.byref(w), layer, seed, block))
    return w


def thresholds_materialize(rule, n, step_t, *, weyl=None, sr_seed=0, layer=0, first_flat=0):
    """Test aid: the 24-bit thresholds of `n` consecutive entries as a CUDA uint32 tensor (as int32 storage)."""
    import torch
    out = torch.empty(n, dtype=torch.int32, device="cuda")
    wp = ctypes.byref(weyl) if weyl is not None else None
    _check(lib().ssdq_thresholds_materialize(rule, wp, sr_seed, layer, first_flat, n, step_t & 0xFFFFFFFF, _ptr(out), _stream()))
    return out


def make_desc(state, scales, fmt, *, A, D, rule, weyl=None, sr_seed=0, layer=0, scale_block=0, batch_index_base=0,
              x=None, dt=None, Bm=None, Cm=None, y=None, dt_bias=None, dt_softplus=False, ngroups=1, z=None,
              head_index_base=0, nheads_global=0) -> UpdateDesc:
    """Describe one layer's problem.  `state` is a CUDA tensor of shape [B, H, P, N] holding the codes
    (uint8 for E4M3, int16/uint16/float16/bfloat16 for the 16-bit formats, float32 for the FP32 twin)."""
    B, H, P, N = state.shape
    d = UpdateDesc()
    d.batch, d.nheads, d.headdim, d.dstate = B, H, P, N
    d.state, d.scales, d.scale_block, d.format = _ptr(state), _ptr(scales), scale_block, fmt
    d.x, d.dt, d.A, d.Bm, d.Cm, d.D = _ptr(x), _ptr(dt), _ptr(A), _ptr(Bm), _ptr(Cm), _ptr(D)
    d.a_per_state = int(A.dim() == 2)
    d.y = _ptr(y)
    d.rule = rule
    if weyl is not None:
        d.weyl = weyl
    d.sr_seed, d.layer, d.batch_index_base = sr_seed, layer, batch_index_base
    d.dt_bias, d.z, d.dt_softplus, d.ngroups = _ptr(dt_bias), _ptr(z), int(bool(dt_softplus)), ngroups
    d.head_index_base, d.nheads_global = head_index_base, nheads_global
    # keep the tensors alive as long as the descriptor
    d._keep = (state, scales, A, D, x, dt, Bm, Cm, y, dt_bias, z)
    return d


def ssd_state_update(desc: UpdateDesc, step_t: int, *, x=None, dt=None, Bm=None, Cm=None, y=None, z=None):
    """One fused decode step of one layer, in place on desc.state; y is written.  Per-step tensors may be
    given here (they overwrite the descriptor's pointers)."""
    if x is not None:
        desc.x, desc.dt, desc.Bm, desc.Cm, desc.y = _ptr(x), _ptr(dt), _ptr(Bm), _ptr(Cm), _ptr(y)
        desc.z = _ptr(z)
    _check(lib().ssd_state_update(ctypes.byref(desc), step_t & 0xFFFFFFFF, _stream()))


def quantize_store(src, codes, scales, fmt, rule, step_t, *, weyl=None, sr_seed=0, layer=0, scale_block=0,
                   row_index_base=0):
    """Quantise float32 CUDA tensor `src` [n_rows, row_len] into `codes` (and `scales` for E4M3)."""
    n_rows, row_len = src.shape
    wp = ctypes.byref(weyl) if weyl is not None else None
    _check(lib().quantize_store(_ptr(src), _ptr(codes), _ptr(scales), n_rows, row_len, scale_block, fmt, rule, wp,
                                sr_seed, layer, row_index_base, step_t & 0xFFFFFFFF, _stream()))


def dequantize(codes, scales, fmt, out, scale_block=0):
    _check(lib().ssdq_dequantize(_ptr(codes), _ptr(scales), codes.numel(), fmt, scale_block, _ptr(out), _stream()))


def make_step_inputs(x, dt, Bm, Cm, y, z=None) -> StepInputs:
    """x [ring, L, B, H, P], dt [ring, L, B, H], Bm/Cm [ring, L, B, (G,) N], y and optional gate z [ring, L, B, H, P];
    float32, all on the device or (for ssd_decode_run_host's host side) all pinned host tensors."""
    s = StepInputs()
    s.ring = x.shape[0]
    s.x, s.stride_x = _ptr(x), x[0, 0].numel()
    s.dt, s.stride_dt = _ptr(dt), dt[0, 0].numel()
    s.Bm, s.stride_B = _ptr(Bm), Bm[0, 0].numel()
    s.Cm, s.stride_C = _ptr(Cm), Cm[0, 0].numel()
    s.y, s.stride_y = _ptr(y), y[0, 0].numel()
    if z is not None:
        s.z, s.stride_z = _ptr(z), z[0, 0].numel()
    s._keep = (x, dt, Bm, Cm, y, z)
    return s


def ssd_decode_run(layer_descs, t_first: int, n_steps: int, step_inputs: StepInputs):
    """n_steps decode steps over all layers on the current stream (one launch per layer per step)."""
    arr = (UpdateDesc * len(layer_descs))(*layer_descs)
    _check(lib().ssd_decode_run(arr, len(layer_descs), t_first & 0xFFFFFFFF, n_steps, ctypes.byref(step_inputs), _stream()))


def state_error(codes, scales, twin, fmt, scale_block=0, workspace=None):
    """Per-head sums (err2, ref2) of (dequant(codes) - twin)^2 and twin^2 as CUDA float64 tensors [H].
    codes [B,H,P,N]; twin float32 [B,H,P,N].  `workspace` (uint8 CUDA tensor) is allocated here if not given."""
    import torch
    B, H, P, N = codes.shape
    need = int(lib().ssdq_state_error_workspace_bytes(B, H))
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=codes.device)
    err2 = torch.empty(H, dtype=torch.float64, device=codes.device)
    ref2 = torch.empty(H, dtype=torch.float64, device=codes.device)
    _check(lib().ssdq_state_error(_ptr(codes), _ptr(scales), _ptr(twin), B, H, P, N, fmt, scale_block, _ptr(err2), _ptr(ref2),
                                  _ptr(workspace), workspace.numel(), _stream()))
    return err2, ref2


STATE_ERROR_STATIC_MAX_ITEMS = 65536


def state_error_static(codes, scales, twin, fmt, err2, ref2, scale_block=0):
    """ssdq_state_error_static: the per-head state-error sums written into the caller's float64 CUDA tensors
    `err2`, `ref2` [H] without any device allocation -- the scratch is a fixed 1 MiB array inside the library, so
    batch * nheads may not exceed STATE_ERROR_STATIC_MAX_ITEMS, calls on one device must not overlap, and the
    first call on a device should come before any stream capture.  For callers (a serving process whose pool
    owns all of HBM, a hook inside the decode loop) that cannot call cudaMalloc."""
    B, H, P, N = codes.shape
    _check(lib().ssdq_state_error_static(_ptr(codes), _ptr(scales), _ptr(twin), B, H, P, N, fmt, scale_block,
                                         _ptr(err2), _ptr(ref2), _stream()))


def readout_kl(y_ref, y_q):
    """KL(softmax(y_ref[b]) || softmax(y_q[b])) per sequence; y_* float32 CUDA tensors [B, ...]."""
    import torch
    B = y_ref.shape[0]
    out = torch.empty(B, dtype=torch.float32, device=y_ref.device)
    _check(lib().ssdq_readout_kl(_ptr(y_ref), _ptr(y_q), B, y_ref[0].numel(), _ptr(out), _stream()))
    return out


def ssd_decode_run_host(layer_descs, t_first: int, n_steps: int, host_io: StepInputs, staging: StepInputs):
    """n_steps decode steps with per-step inputs in (pinned) HOST tensors and y returned to HOST tensors, copies
    overlapped with compute.  `host_io` and `staging` come from make_step_inputs on host and device tensors of
    identical per-slot shapes; staging needs 2 to 8 ring slots.  Synchronise the current stream before reading y."""
    arr = (UpdateDesc * len(layer_descs))(*layer_descs)
    _check(lib().ssd_decode_run_host(arr, len(layer_descs), t_first & 0xFFFFFFFF, n_steps, ctypes.byref(host_io),
                                     ctypes.byref(staging), _stream()))


def replay_step(w, decay, rows_per_decay, codes, scales, fmt, rule, step_t, *, weyl=None, sr_seed=0, layer=0, scale_block=0,
                row_index_base=0):
    """Open-loop replay h <- Q(decay * h + w) in place on `codes` [n_rows, row_len] (and `scales`)."""
    n_rows, row_len = codes.shape
    wp = ctypes.byref(weyl) if weyl is not None else None
    _check(lib().ssd_replay_step(_ptr(w), _ptr(decay), rows_per_decay, _ptr(codes), _ptr(scales), n_rows, row_len, scale_block,
                                 fmt, rule, wp, sr_seed, layer, row_index_base, step_t & 0xFFFFFFFF, _stream()))


def ssd_decode_run_checkpointed(layer_descs, work_states, every: int, t_first: int, n_steps: int, step_inputs: StepInputs):
    """Decode with the state in FP32 between checkpoints; every `every`-th write is rounded into each layer's store.
    work_states: one float32 CUDA tensor [B, H, P, N] per layer."""
    arr = (UpdateDesc * len(layer_descs))(*layer_descs)
    ptrs = (_vp * len(work_states))(*[w.data_ptr() for w in work_states])
    _check(lib().ssd_decode_run_checkpointed(arr, ptrs, len(layer_descs), every, t_first & 0xFFFFFFFF, n_steps,
                                             ctypes.byref(step_inputs), _stream()))


class DecodeGraph:
    """A replayable CUDA graph of `steps_per_launch` decode steps over all layers (ssd_decode_graph_*).  The write index
    lives in `step_counter`, a CUDA int32 tensor of one element that each replay advances by steps_per_launch."""

    def __init__(self, layer_descs, steps_per_launch: int, step_inputs: StepInputs, step_counter):
        self._keep = (layer_descs, step_inputs, step_counter)
        arr = (UpdateDesc * len(layer_descs))(*layer_descs)
        self.handle = _vp()
        _check(lib().ssd_decode_graph_create(ctypes.byref(self.handle), arr, len(layer_descs), steps_per_launch,
                                             ctypes.byref(step_inputs), _ptr(step_counter)))

    def launch(self):
        _check(lib().ssd_decode_graph_launch(self.handle, _stream()))

    def close(self):
        if self.handle:
            lib().ssd_decode_graph_destroy(self.handle)
            self.handle = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def copy(src, dst):
    """ssdq_copy: plain 128-bit copy of `src` into `dst` (same byte size) by the library's copy kernel -- the floor of
    the timing protocol."""
    nbytes = src.numel() * src.element_size()
    assert nbytes == dst.numel() * dst.element_size()
    _check(lib().ssdq_copy(_ptr(src), _ptr(dst), nbytes, _stream()))


def last_kernel() -> str:
    return lib().ssdq_last_kernel().decode()


def launch_count() -> int:
    return int(lib().ssdq_launch_count())


def set_launch_overlap(enabled: bool) -> bool:
    """Programmatic dependent launch between the drivers' own kernels (on by default); returns the previous setting."""
    return bool(lib().ssdq_set_launch_overlap(int(bool(enabled))))

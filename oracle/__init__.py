"""CPU oracle of the quantized selective-state-update decode step -- TEST INFRASTRUCTURE ONLY.

A thin ctypes wrapper over ``ssdq_oracle.cpp`` (plain C++17, compiled on first use with g++).
Nothing in the product package imports this module; it serves the tests, the smoke check and the
CPU-baseline leg of the benchmark.  It shares no code with the CUDA path.

Every function mirrors one exported symbol of the C++ file; see that file for the passages of the
paper each step follows (Eq. 1, Eq. 2, Appendix B "Formats" and "Dithers").
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

FP16, BF16, E4M3, FP32 = 0, 1, 2, 3
INT8, INT7, INT6, INT4 = 4, 5, 6, 7          # symmetric block-absmax integers, one int8 per entry
INT_QMAX = {INT8: 127, INT7: 63, INT6: 31, INT4: 7}
RTN, SR, WEYL, SR_HASH = 0, 1, 2, 3
FORMAT_NAMES = {FP16: "fp16", BF16: "bf16", E4M3: "e4m3", FP32: "fp32", INT8: "int8", INT7: "int7", INT6: "int6", INT4: "int4"}
RULE_NAMES = {RTN: "rtn", SR: "sr", WEYL: "weyl", SR_HASH: "sr_hash"}
CODE_DTYPE = {FP16: np.uint16, BF16: np.uint16, E4M3: np.uint8, FP32: np.uint32, INT8: np.uint8, INT7: np.uint8,
              INT6: np.uint8, INT4: np.uint8}


def has_block_scale(fmt):
    return fmt == E4M3 or fmt in INT_QMAX

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ssdq_oracle.cpp")
_LIB = os.path.join(_HERE, "libssdq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (g++, no fast-math, no FMA contraction).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u32, u64, f32, i32 = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_float, ctypes.c_int
        vp = ctypes.c_void_p
        L.oracle_weyl_acc.restype = u32
        L.oracle_weyl_acc.argtypes = [u32] * 5
        L.oracle_philox4x32_10.restype = None
        L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
        L.oracle_exp_spec.restype = f32
        L.oracle_exp_spec.argtypes = [f32]
        L.oracle_fmix32.restype = u32
        L.oracle_fmix32.argtypes = [u32]
        L.oracle_round.restype = f32
        L.oracle_round.argtypes = [f32, i32, i32, u32]
        L.oracle_encode.restype = u32
        L.oracle_encode.argtypes = [f32, i32]
        L.oracle_decode.restype = f32
        L.oracle_decode.argtypes = [u32, i32]
        L.oracle_threshold.restype = u32
        L.oracle_threshold.argtypes = [i32, u32, u32, u32, u64, u64, u32]
        L.oracle_round_array.restype = None
        L.oracle_round_array.argtypes = [vp, vp, u64, i32, i32, vp]
        L.oracle_round_encode_array.restype = None
        L.oracle_round_encode_array.argtypes = [vp, vp, u64, u64, i32, i32, vp]
        L.oracle_exp_spec_array.restype = None
        L.oracle_exp_spec_array.argtypes = [vp, u64, vp]
        L.oracle_state_update.restype = i32
        L.oracle_state_update.argtypes = [vp, vp, i32, u32, u32, u32, u32, u32, vp, vp, vp, i32, vp, vp, vp, vp,
                                          i32, u32, u32, u32, u64, u32, u32, vp, i32, u32, vp, u32, u32]
        L.oracle_softplus_spec.restype = f32
        L.oracle_softplus_spec.argtypes = [f32]
        L.oracle_block_scale_array.restype = None
        L.oracle_block_scale_array.argtypes = [vp, u64, i32, vp]
        L.oracle_softplus_spec_array.restype = None
        L.oracle_softplus_spec_array.argtypes = [vp, u64, vp]
        L.oracle_quantize_store.restype = i32
        L.oracle_quantize_store.argtypes = [vp, vp, vp, u64, u32, i32, u32, i32, u32, u32, u32, u64, u64, u32]
        L.oracle_replay_step.restype = i32
        L.oracle_replay_step.argtypes = [vp, vp, u32, vp, vp, u64, u32, i32, u32, i32, u32, u32, u32, u64, u64, u32]
        L.oracle_dequantize.restype = None
        L.oracle_dequantize.argtypes = [vp, vp, u64, i32, u32, vp]
        L.oracle_num_threads.restype = i32
        L.oracle_num_threads.argtypes = []
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


# ---- elementary functions -------------------------------------------------------------------
def weyl_acc(r, c, layer, seed, t) -> int:
    m = 0xFFFFFFFF
    return lib().oracle_weyl_acc(r & m, c & m, layer & m, seed & m, t & m)


def weyl_u24(r, c, layer, seed, t) -> int:
    return weyl_acc(r, c, layer, seed, t) >> 8


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def fmix32(h) -> int:
    return lib().oracle_fmix32(h & 0xFFFFFFFF)


def exp_spec(z):
    z = _f32(np.atleast_1d(z))
    out = np.empty_like(z)
    lib().oracle_exp_spec_array(_ptr(z), z.size, _ptr(out))
    return out


def threshold(rule, flat, t, layer=0, weyl_seed=0, weyl_block=16, sr_seed=0) -> int:
    return lib().oracle_threshold(rule, layer, weyl_seed, weyl_block, sr_seed, flat, t & 0xFFFFFFFF)


def thresholds(rule, flats, t, layer=0, weyl_seed=0, weyl_block=16, sr_seed=0):
    return np.array([threshold(rule, int(f), t, layer, weyl_seed, weyl_block, sr_seed) for f in flats],
                    dtype=np.uint32)


def round_values(v, U, fmt, rule):
    """Eq. 2 on the local grid of `fmt`, elementwise; returns the rounded values as float32."""
    v = _f32(np.atleast_1d(v))
    U = np.ascontiguousarray(np.broadcast_to(np.asarray(U, dtype=np.uint32), v.shape))
    out = np.empty_like(v)
    lib().oracle_round_array(_ptr(v), _ptr(U), v.size, fmt, rule, _ptr(out))
    return out


def round_encode(v, U, fmt, rule):
    """Codes of Eq. 2 applied to every entry of float32 `v` with thresholds `U` (an array like v, one integer for
    all entries, or None under RTN): encode(round_values(v, U)) in one parallel pass."""
    v = _f32(v)
    codes = np.empty(v.shape, dtype=CODE_DTYPE[fmt])
    if U is None:
        Ua, nU = None, 0
    else:
        Ua = np.ascontiguousarray(np.atleast_1d(U), dtype=np.uint32)
        nU = Ua.size
        assert nU in (1, v.size)
    lib().oracle_round_encode_array(_ptr(v), _ptr(Ua), nU, v.size, fmt, rule, _ptr(codes))
    return codes


def encode(q, fmt):
    q = _f32(np.atleast_1d(q))
    return np.array([lib().oracle_encode(float(x), fmt) for x in q.ravel()],
                    dtype=CODE_DTYPE[fmt]).reshape(q.shape)


def decode(codes, fmt):
    codes = np.atleast_1d(codes)
    return np.array([lib().oracle_decode(int(c), fmt) for c in codes.ravel()],
                    dtype=np.float32).reshape(codes.shape)


# ---- the decode step ------------------------------------------------------------------------
def softplus_spec(x):
    x = _f32(np.atleast_1d(x))
    out = np.empty_like(x)
    lib().oracle_softplus_spec_array(_ptr(x), x.size, _ptr(out))
    return out


def block_scale(amax, fmt):
    """FP32 block scale max(amax / top, FLT_MIN) of a scaled store (top = 448 for E4M3, q_max for INTb), elementwise."""
    amax = _f32(np.atleast_1d(amax))
    out = np.empty_like(amax)
    lib().oracle_block_scale_array(_ptr(amax), amax.size, fmt, _ptr(out))
    return out


def state_update(state, scales, fmt, scale_block, x, dt, A, Bm, Cm, D, rule, step_t, *, layer=0,
                 weyl_seed=0, weyl_block=16, sr_seed=0, batch_index_base=0, dt_bias=None, dt_softplus=False,
                 ngroups=1, z=None, head_index_base=0, nheads_global=0):
    """One decode step of one layer, in place on `state` (and `scales`).  Returns y [B,H,P] float32.

    state [B,H,P,N] of CODE_DTYPE[fmt] (float32 viewed as uint32 for FP32); x [B,H,P]; dt [B,H];
    A [H] or [H,N]; Bm, Cm [B,N] (or [B,G,N] with ngroups=G); D [H] or None; dt_bias [H] or None; with
    dt_softplus the step size is softplus_spec(dt + dt_bias); z [B,H,P] or None gates y by z * sigmoid(z).
    The arrays may hold a slice of the layer: sequences from batch_index_base on, heads from head_index_base on out of
    nheads_global (0 = H); the thresholds are drawn at the entry's index in the whole layer.
    """
    Bsz, H, P, N = state.shape
    assert state.flags.c_contiguous and state.dtype == CODE_DTYPE[fmt]
    x, dt, A, Bm, Cm = _f32(x), _f32(dt), _f32(A), _f32(Bm), _f32(Cm)
    D = None if D is None else _f32(D)
    gshape = (Bsz, N) if ngroups == 1 else (Bsz, ngroups, N)
    assert x.shape == (Bsz, H, P) and dt.shape == (Bsz, H) and Bm.shape == gshape and Cm.shape == gshape
    dt_bias = None if dt_bias is None else _f32(dt_bias)
    z = None if z is None else _f32(z)
    a_per_state = int(A.ndim == 2)
    assert A.shape == ((H, N) if a_per_state else (H,))
    y = np.empty((Bsz, H, P), dtype=np.float32)
    if scales is not None:
        assert scales.dtype == np.float32 and scales.flags.c_contiguous
    rc = lib().oracle_state_update(_ptr(state), _ptr(scales), fmt, scale_block, Bsz, H, P, N, _ptr(x), _ptr(dt),
                                   _ptr(A), a_per_state, _ptr(Bm), _ptr(Cm), _ptr(D), _ptr(y), rule, layer,
                                   weyl_seed, weyl_block, sr_seed, batch_index_base, step_t, _ptr(dt_bias),
                                   int(bool(dt_softplus)), ngroups, _ptr(z), head_index_base, nheads_global)
    if rc != 0:
        raise ValueError("oracle_state_update: undefined argument combination")
    return y


def quantize_store(src, fmt, rule, step_t, *, scale_block=0, layer=0, weyl_seed=0, weyl_block=16, sr_seed=0,
                   row_index_base=0):
    """Quantise float32 `src` [n_rows, row_len]; returns (codes, scales or None)."""
    src = _f32(src)
    n_rows, row_len = src.shape
    codes = np.zeros((n_rows, row_len), dtype=CODE_DTYPE[fmt])
    scales = np.zeros((n_rows, row_len // scale_block), dtype=np.float32) if has_block_scale(fmt) else None
    rc = lib().oracle_quantize_store(_ptr(src), _ptr(codes), _ptr(scales), n_rows, row_len, fmt, scale_block, rule,
                                     layer, weyl_seed, weyl_block, sr_seed, row_index_base, step_t)
    if rc != 0:
        raise ValueError("oracle_quantize_store: undefined argument combination")
    return codes, scales


def replay_step(w, a, rows_per_decay, codes, scales, fmt, rule, step_t, *, scale_block=0, layer=0, weyl_seed=0,
                weyl_block=16, sr_seed=0, row_index_base=0):
    """Open-loop replay h <- Q(a h + w), in place on codes [n_rows, row_len] (and scales); w float32 [n_rows, row_len],
    a float32 [n_rows / rows_per_decay]."""
    w, a = _f32(w), _f32(a)
    n_rows, row_len = codes.shape
    assert w.shape == codes.shape and a.size * rows_per_decay == n_rows and codes.flags.c_contiguous
    rc = lib().oracle_replay_step(_ptr(w), _ptr(a), rows_per_decay, _ptr(codes), _ptr(scales), n_rows, row_len, fmt, scale_block,
                                  rule, layer, weyl_seed, weyl_block, sr_seed, row_index_base, step_t)
    if rc != 0:
        raise ValueError("oracle_replay_step: undefined argument combination")


def dequantize(codes, scales, fmt, scale_block=0):
    codes = np.ascontiguousarray(codes)
    out = np.empty(codes.shape, dtype=np.float32)
    lib().oracle_dequantize(_ptr(codes), _ptr(scales), codes.size, fmt, max(scale_block, 1), _ptr(out))
    return out


def new_state(shape, fmt, scale_block=0):
    """All-zero state (h_0 = 0) and its scale array (E4M3: scale of an all-zero block)."""
    Bsz, H, P, N = shape
    state = np.zeros(shape, dtype=CODE_DTYPE[fmt])
    scales = None
    if has_block_scale(fmt):
        n_scales = Bsz * H if scale_block == P * N and scale_block != N else Bsz * H * P * (N // scale_block)
        scales = np.full(n_scales, np.finfo(np.float32).tiny, dtype=np.float32)
    return state, scales


def num_threads() -> int:
    return lib().oracle_num_threads()


# ---- sanity metrics (plain definitions, float64) ---------------------------------------------
def state_error_per_head(codes, scales, twin, fmt, scale_block=0):
    """Appendix B "Open-loop replay": sum (h_hat - h)^2 and sum h^2, here kept per head.
    codes [B,H,P,N]; twin float32 [B,H,P,N].  Returns (err2 [H], ref2 [H]) float64."""
    hq = dequantize(codes, scales, fmt, scale_block).astype(np.float64).reshape(codes.shape)
    ref = np.asarray(twin, dtype=np.float64).reshape(codes.shape)
    return ((hq - ref) ** 2).sum(axis=(0, 2, 3)), (ref ** 2).sum(axis=(0, 2, 3))


def readout_kl(y_ref, y_q):
    """KL(p || q) = sum p log(p / q) per sequence with p, q the softmax of each sequence's readout vector
    (the per-token KL of Section 4 "What we measure", on a surrogate distribution)."""
    a = np.asarray(y_ref, dtype=np.float64).reshape(len(y_ref), -1)
    b = np.asarray(y_q, dtype=np.float64).reshape(len(y_q), -1)
    lp = a - a.max(axis=1, keepdims=True)
    lp = lp - np.log(np.exp(lp).sum(axis=1, keepdims=True))
    lq = b - b.max(axis=1, keepdims=True)
    lq = lq - np.log(np.exp(lq).sum(axis=1, keepdims=True))
    return (np.exp(lp) * (lp - lq)).sum(axis=1)

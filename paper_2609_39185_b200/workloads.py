"""Seeded synthetic decode workloads (input data only -- none of the method's arithmetic lives here).

The five named configurations are shaped like the Mamba and hybrid decode workloads the paper
measures on (Mamba-1 state [d_inner, 16] per sequence, Mamba-2 / hybrid heads of 64 x 128,
Appendix B "Models and assets" and "Runners"); the paper's datasets and trained weights are not
available, so seeded random inputs with the same shapes and a spread of decay time constants
(Section 2: most entries short-memory, a minority with tau >= 100 or >= 1000) stand in for them.

Both the CUDA library and the CPU oracle consume the arrays produced here; neither is imported.
numpy's counter-based ``default_rng`` is keyed by (config, seed, layer, step, tensor), so any
(layer, step) can be generated on its own and a slice of the batch can be compared exactly.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import numpy as np

FP16, BF16, E4M3, FP32 = 0, 1, 2, 3
INT8, INT7, INT6, INT4 = 4, 5, 6, 7
SCALED_FORMATS = (E4M3, INT8, INT7, INT6, INT4)
RTN, SR, WEYL, SR_HASH = 0, 1, 2, 3
FORMAT_NAMES = {FP16: "fp16", BF16: "bf16", E4M3: "e4m3", FP32: "fp32", INT8: "int8", INT7: "int7", INT6: "int6", INT4: "int4"}
RULE_NAMES = {RTN: "rtn", SR: "sr", WEYL: "weyl", SR_HASH: "sr_hash"}
CODE_BYTES = {FP16: 2, BF16: 2, E4M3: 1, FP32: 4, INT8: 1, INT7: 1, INT6: 1, INT4: 1}

_T_A, _T_D, _T_X, _T_DT, _T_B, _T_C, _T_H0 = range(7)


@dataclass(frozen=True)
class DecodeConfig:
    name: str
    index: int          # 1-based number of the configuration
    batch: int
    nheads: int
    headdim: int
    dstate: int
    fmt: int
    steps: int          # decode horizon T
    n_layers: int = 1
    weyl_block: int = 16    # entries per dither block along N (16 for Mamba-shaped, N for hybrid-shaped)
    scale_block: int = 0    # E4M3 only: entries per FP32 scale
    a_per_state: bool = False   # Mamba-1: A is [H, N]
    recipe: str = "mamba2"

    @property
    def state_shape(self):
        return (self.batch, self.nheads, self.headdim, self.dstate)

    @property
    def entries_per_layer(self):
        return self.batch * self.nheads * self.headdim * self.dstate

    def state_bytes_per_layer(self):
        n = self.entries_per_layer
        b = n * CODE_BYTES[self.fmt]
        if self.fmt in SCALED_FORMATS:
            b += 4 * n // self.scale_block
        return b

    def algorithmic_bytes_per_layer_step(self):
        """Bytes one fused update of one layer must move: state (+scales) read and written, x in,
        y out, dt, B, C, A, D in."""
        B, H, P, N = self.state_shape
        a_elems = H * N if self.a_per_state else H
        return 2 * self.state_bytes_per_layer() + 4 * (2 * B * H * P + B * H + 2 * B * N + a_elems + H)

    def with_batch(self, batch):
        return replace(self, batch=batch)


CONFIGS = {
    1: DecodeConfig("tiny-mamba2-fp16", 1, batch=1, nheads=4, headdim=16, dstate=16, fmt=FP16, steps=64,
                    weyl_block=16, recipe="tiny"),
    2: DecodeConfig("mamba1-130m-bf16", 2, batch=8, nheads=1536, headdim=1, dstate=16, fmt=BF16, steps=512,
                    weyl_block=16, a_per_state=True, recipe="mamba1"),
    3: DecodeConfig("mamba2-2.7b-fp16", 3, batch=64, nheads=80, headdim=64, dstate=128, fmt=FP16, steps=256,
                    weyl_block=16, recipe="mamba2"),
    4: DecodeConfig("long-horizon-e4m3", 4, batch=32, nheads=64, headdim=64, dstate=128, fmt=E4M3, steps=4096,
                    weyl_block=128, scale_block=128, recipe="mamba2-slow-heads"),
    5: DecodeConfig("hybrid-stack-bf16", 5, batch=128, nheads=128, headdim=64, dstate=128, fmt=BF16, steps=1024,
                    n_layers=8, weyl_block=128, recipe="mamba2"),
}


def _rng(cfg: DecodeConfig, seed: int, layer: int, step: int, tensor: int):
    return np.random.default_rng([cfg.index, seed, layer, step, tensor])


def _softplus(v):
    return np.logaddexp(0.0, v.astype(np.float64)).astype(np.float32)


def layer_seed(cfg: DecodeConfig, seed: int, layer: int) -> int:
    """Config 5 uses per-layer independent seeds: the layer index is folded into the seed."""
    return seed + layer


def layer_params(cfg: DecodeConfig, layer: int = 0, seed: int = 0):
    """Static per-layer parameters A ([H] or [H, N]) and D ([H]), float32."""
    H, N = cfg.nheads, cfg.dstate
    ra = _rng(cfg, seed, layer, 0, _T_A)
    if cfg.recipe == "tiny":
        A = -np.exp(ra.uniform(0.0, 1.0, H))
    elif cfg.recipe == "mamba1":
        # S4D-real style spectrum -(1..N), broadcast over channels, with +-20 % log-uniform jitter
        A = -(np.arange(1, N + 1, dtype=np.float64)[None, :]) * np.exp(ra.uniform(-0.2, 0.2, (H, N)))
    else:
        A = -np.exp(ra.uniform(-4.0, 1.0, H))
        if cfg.recipe == "mamba2-slow-heads":
            slow = np.arange(H) % 4 == 0      # a quarter of the heads: increments below half an E4M3 step
            A = np.where(slow, -ra.uniform(0.002, 0.02, H), A)
    D = _rng(cfg, seed, layer, 0, _T_D).normal(0.0, 0.1, H)
    return A.astype(np.float32), D.astype(np.float32)


def step_inputs(cfg: DecodeConfig, step: int, layer: int = 0, seed: int = 0, batch_slice=None):
    """Inputs of decode step `step` (1-based) for one layer: x [B,H,P], dt [B,H], Bm, Cm [B,N].

    `batch_slice` (a slice or index array) returns only those sequences; every sequence is drawn
    from its own stream position, so a subset equals the same rows of the full batch.
    """
    B, H, P, N = cfg.state_shape
    f32 = np.float32
    x = _rng(cfg, seed, layer, step, _T_X).standard_normal((B, H, P), dtype=f32)
    g = _rng(cfg, seed, layer, step, _T_DT).standard_normal((B, H), dtype=f32)
    Bm = _rng(cfg, seed, layer, step, _T_B).standard_normal((B, N), dtype=f32)
    Cm = _rng(cfg, seed, layer, step, _T_C).standard_normal((B, N), dtype=f32)
    if cfg.recipe == "tiny":
        dt = _softplus(-2.0 + 0.5 * g)
    elif cfg.recipe == "mamba1":
        dt = _softplus(-3.0 + 0.5 * g)
    else:
        dt = _softplus(-4.0 + 1.0 * g)
        scale = f32(1.0 / np.sqrt(N))
        Bm *= scale
        Cm *= scale
        if cfg.recipe == "mamba2-slow-heads":
            slow = np.arange(H) % 4 == 0
            dt[:, slow] = np.minimum(dt[:, slow], f32(0.05))    # dt * |A| <= 1e-3 on the slow heads
    if batch_slice is not None:
        x, dt, Bm, Cm = x[batch_slice], dt[batch_slice], Bm[batch_slice], Cm[batch_slice]
    return (np.ascontiguousarray(x), np.ascontiguousarray(dt), np.ascontiguousarray(Bm),
            np.ascontiguousarray(Cm))


def initial_state_fp32(cfg: DecodeConfig, layer: int = 0, seed: int = 0, scale: float = 1.0):
    """A full-precision state to quantise as h_0 (the variant in which decode starts from the
    end-of-prefill state instead of zero): N(0, scale^2), float32 [B,H,P,N]."""
    return (scale * _rng(cfg, seed, layer, 0, _T_H0).standard_normal(cfg.state_shape, dtype=np.float32)
            ).astype(np.float32)

"""The seeded workload generators: shapes and sizes of the five named configurations, slicing invariance
(a batch slice equals the same rows of the full batch), and the recipes' ranges."""
import numpy as np

from paper_2609_39185_b200 import workloads as W


def test_named_configurations_have_the_stated_sizes():
    c = W.CONFIGS
    assert c[1].state_shape == (1, 4, 16, 16) and c[1].fmt == W.FP16 and c[1].steps == 64
    assert c[2].state_shape == (8, 1536, 1, 16) and c[2].fmt == W.BF16 and c[2].a_per_state and c[2].steps == 512
    assert c[3].state_shape == (64, 80, 64, 128) and c[3].fmt == W.FP16 and c[3].steps == 256
    assert c[3].state_bytes_per_layer() == 83_886_080                      # "state 84 MB fp16"
    assert c[4].state_shape == (32, 64, 64, 128) and c[4].fmt == W.E4M3 and c[4].steps == 4096 and c[4].scale_block == 128
    assert c[4].state_bytes_per_layer() == 16_777_216 + 4 * 131_072
    assert c[5].state_shape == (128, 128, 64, 128) and c[5].fmt == W.BF16 and c[5].n_layers == 8 and c[5].steps == 1024
    assert c[5].state_bytes_per_layer() * c[5].n_layers == 2_147_483_648   # "~2.1 GB state total"
    assert c[5].algorithmic_bytes_per_layer_step() == 545_457_152
    assert c[5].weyl_block == 128 and c[3].weyl_block == 16                # blocks of 16 for Mamba, N for hybrids


def test_a_batch_slice_equals_the_rows_of_the_full_batch():
    cfg = W.CONFIGS[3].with_batch(6)
    full = W.step_inputs(cfg, 7, layer=2, seed=5)
    part = W.step_inputs(cfg, 7, layer=2, seed=5, batch_slice=slice(2, 5))
    for f, p in zip(full, part):
        assert np.array_equal(f[2:5], p) and p.flags.c_contiguous and p.dtype == np.float32
    again = W.step_inputs(cfg, 7, layer=2, seed=5)
    assert all(np.array_equal(a, b) for a, b in zip(full, again))
    other = W.step_inputs(cfg, 8, layer=2, seed=5)
    assert not np.array_equal(full[0], other[0])


def test_recipes_stay_in_their_ranges():
    for idx in (1, 2, 3, 4):
        cfg = W.CONFIGS[idx].with_batch(2)
        A, D = W.layer_params(cfg)
        assert np.all(A < 0) and A.dtype == np.float32 and D.shape == (cfg.nheads,)
        assert A.shape == ((cfg.nheads, cfg.dstate) if cfg.a_per_state else (cfg.nheads,))
        x, dt, Bm, Cm = W.step_inputs(cfg, 1)
        assert np.all(dt > 0) and np.all(np.isfinite(x)) and Bm.shape == (2, cfg.dstate)
    cfg = W.CONFIGS[4].with_batch(2)
    A, _ = W.layer_params(cfg)
    _, dt, _, _ = W.step_inputs(cfg, 3)
    slow = np.arange(cfg.nheads) % 4 == 0
    assert np.all(dt[:, slow] * np.abs(A[slow]) <= 1e-3 + 1e-9)            # increments below half an E4M3 step
    assert slow.mean() == 0.25
    A2, _ = W.layer_params(W.CONFIGS[2])
    ratio = -A2 / np.arange(1, 17)[None, :]
    assert np.all(ratio > np.exp(-0.2) - 1e-6) and np.all(ratio < np.exp(0.2) + 1e-6)
    a5 = [W.layer_params(W.CONFIGS[5], l, W.layer_seed(W.CONFIGS[5], 0, l))[0] for l in (0, 1)]
    assert not np.array_equal(a5[0], a5[1])                                # per-layer independent seeds

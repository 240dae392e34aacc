"""GPU parity of the fused decode step (through the C ABI) against the CPU oracle: stored state bit
for bit, y within 1e-5 of the absolute-sum scale, on the five named workloads and on edge shapes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39185_b200 import ssdq, workloads
from parity import Pair, run_parity, to_dev, codes_to_dev, codes_to_host

pytestmark = pytest.mark.gpu

RULES = [ssdq.RTN, ssdq.SR, ssdq.WEYL, ssdq.SR_HASH]
CFG = workloads.CONFIGS


@pytest.mark.parametrize("rule", RULES)
def test_config1_tiny_fp16_full_horizon(rule):
    run_parity(CFG[1], rule, CFG[1].steps)


@pytest.mark.parametrize("rule", RULES)
def test_config2_mamba1_bf16_full_horizon(rule):
    run_parity(CFG[2], rule, CFG[2].steps, check_every=16)


@pytest.mark.parametrize("rule", RULES)
def test_config3_mamba2_fp16_full_size_few_steps(rule):
    run_parity(CFG[3], rule, 3)


@pytest.mark.parametrize("rule", RULES)
def test_config3_full_horizon_on_a_batch_slice(rule):
    # sequences are independent: the last two sequences, addressed with their global batch index
    run_parity(CFG[3], rule, CFG[3].steps, batch_slice=slice(62, 64), batch_index_base=62, check_every=32)


@pytest.mark.parametrize("rule", RULES)
def test_config4_e4m3_full_size_few_steps(rule):
    run_parity(CFG[4], rule, 4)


@pytest.mark.parametrize("rule", RULES)
def test_config4_full_horizon_on_one_sequence(rule):
    # all 4096 quantised steps (the slow heads' increments stay below half an E4M3 step throughout)
    run_parity(CFG[4], rule, CFG[4].steps, batch_slice=slice(31, 32), batch_index_base=31, check_every=256)


@pytest.mark.parametrize("rule", RULES)
def test_config5_full_horizon_on_the_last_two_sequences(rule):
    # layer 7 with its own seed, all 1024 steps, sequences 126 and 127 addressed by their global index
    cfg = CFG[5]
    run_parity(cfg, rule, cfg.steps, layer=7, seed=workloads.layer_seed(cfg, 0, 7), batch_slice=slice(126, 128),
               batch_index_base=126, sr_seed=7, check_every=128)


@pytest.mark.parametrize("rule", RULES)
def test_config5_full_batch_launch_sampled_sequences(rule):
    """The launch configuration the benchmark times (B=128, H=128, P=64, N=128, bf16): every one of the 8 layers with
    its own seed, 8 steps at full batch; the oracle recomputes sequences 0, 1, 126, 127 (sequences are independent, so
    its cost is per sampled sequence) and only those are read back."""
    from parity import y_close
    cfg = CFG[5]
    steps = 8
    for layer in range(cfg.n_layers):
        seed = workloads.layer_seed(cfg, 0, layer)
        A, D = workloads.layer_params(cfg, layer, seed)
        gpu = Pair(cfg.state_shape, cfg.fmt, rule, A, D, weyl_block=cfg.weyl_block, layer=layer, sr_seed=seed)
        subs = {b0: Pair((2,) + cfg.state_shape[1:], cfg.fmt, rule, A, D, weyl_block=cfg.weyl_block, layer=layer,
                         sr_seed=seed, batch_index_base=b0) for b0 in (0, 126)}
        for t in range(1, steps + 1):
            x, dt, Bm, Cm = workloads.step_inputs(cfg, t, layer, seed)
            y_d = gpu.step_gpu(t, x, dt, Bm, Cm)
            for b0, sub in subs.items():
                sl = slice(b0, b0 + 2)
                y_ref = sub.step_oracle(t, x[sl], dt[sl], Bm[sl], Cm[sl])
                got = codes_to_host(gpu.state_d[sl].contiguous(), cfg.fmt)
                assert np.array_equal(got, sub.state_h), (layer, t, b0)
                new_f32 = oracle.dequantize(sub.state_h, None, cfg.fmt).reshape(sub.shape)
                ok, worst = y_close(y_d[sl].cpu().numpy(), y_ref, Cm[sl], new_f32, D, x[sl])
                assert ok, (layer, t, b0, worst)
        del gpu
        torch.cuda.empty_cache()


@pytest.mark.parametrize("rule", RULES)
@pytest.mark.parametrize("fmt", [ssdq.INT8, ssdq.INT4])
def test_int_store_on_the_hybrid_shape(rule, fmt):
    """The paper's headline format (INT8, FP32 block scale, block = state dimension for the hybrids) on the
    config 4 shape: full size for a few steps, then a long horizon on one sequence."""
    from dataclasses import replace
    cfg = replace(CFG[4], fmt=fmt)
    run_parity(cfg, rule, 3)
    run_parity(cfg, rule, 512, batch_slice=slice(5, 6), batch_index_base=5, check_every=64)


@pytest.mark.parametrize("rule", RULES)
def test_int8_store_on_the_mamba1_shape(rule):
    from dataclasses import replace
    cfg = replace(CFG[2], fmt=ssdq.INT8, scale_block=16)      # blocks of 16 entries for the Mamba models
    run_parity(cfg, rule, 64, check_every=8)


@pytest.mark.parametrize("fmt", [ssdq.E4M3, ssdq.INT8, ssdq.INT4])
@pytest.mark.parametrize("rule", RULES)
@pytest.mark.parametrize("shape", [(2, 3, 64, 128), (1, 2, 128, 128), (3, 2, 32, 128), (1, 2, 64, 256), (2, 2, 64, 64)])
def test_one_scale_per_head(fmt, rule, shape):
    """scale_block = P * N: a single FP32 scale per (sequence, head), from the maximum over the whole head (the reading
    of "per-head scale"); codes and scales bit for bit, from the zero state and over several writes."""
    B, H, P, N = shape
    rng = np.random.default_rng(hash((fmt, rule) + shape) % 2**32)
    f32 = np.float32
    A = -np.exp(rng.uniform(-4, 1, H)).astype(f32)
    D = rng.normal(0, 0.1, H).astype(f32)
    pair = Pair(shape, fmt, rule, A, D, weyl_block=N if P % 64 else 16, scale_block=P * N, layer=2, weyl_seed=1, sr_seed=777,
                batch_index_base=9)
    assert pair.scales_h.shape == (B * H,)
    for t in range(1, 6):
        x = rng.standard_normal((B, H, P)).astype(f32)
        if t == 3:
            x[0, 0] = 0.0                                                      # a head that only decays on this step
        dt = np.log1p(np.exp(rng.normal(-2, 1, (B, H)))).astype(f32)
        Bm = rng.standard_normal((B, N)).astype(f32)
        Cm = rng.standard_normal((B, N)).astype(f32)
        # the y tolerance is relative to sum_n |C_n h'_n| + |D x| of the UNROUNDED h': with one scale for the whole head the
        # stored state rounds small entries to zero and no longer gives that scale, so it is computed here in float64
        h_prev = oracle.dequantize(pair.state_h, pair.scales_h, fmt, P * N).reshape(shape).astype(np.float64)
        a = np.exp(dt.astype(np.float64) * A[None, :])
        h_new = a[:, :, None, None] * h_prev + (dt.astype(np.float64)[:, :, None] * x)[..., None] * Bm.astype(np.float64)[:, None, None, :]
        absum = np.einsum("bhpn,bn->bhp", np.abs(h_new), np.abs(Cm.astype(np.float64))) + np.abs(D.astype(np.float64))[None, :, None] * np.abs(x)
        pair.step_gpu(t, x, dt, Bm, Cm)
        y_ref = pair.step_oracle(t, x, dt, Bm, Cm)
        pair.compare(t, x, dt, Bm, Cm, y_ref, y_absum=absum)
    assert ssdq.last_kernel() == "ssd_update_headscale_kernel"


def test_one_scale_per_head_on_the_config4_shape_full_size():
    from dataclasses import replace
    cfg = replace(CFG[4], scale_block=CFG[4].headdim * CFG[4].dstate)
    run_parity(cfg, ssdq.WEYL, 3)
    run_parity(replace(cfg, fmt=ssdq.INT8), ssdq.WEYL, 3)


SHAPES = [
    # (B, H, P, N, a_per_state)
    (1, 1, 1, 16, False), (3, 5, 7, 16, True), (2, 3, 64, 128, False), (5, 7, 3, 128, False), (2, 2, 100, 64, False),
    (1, 9, 8, 256, False), (2, 130, 1, 32, True), (1, 3, 65, 128, True), (4, 1, 16, 64, True),
    # heads the tile kernel takes with 16, 2 and 4 rows per slot
    (2, 3, 128, 128, False), (1, 2, 64, 256, False), (2, 3, 32, 128, False), (2, 2, 64, 64, False), (2, 2, 32, 64, False),
]


@pytest.mark.parametrize("fmt", [ssdq.FP16, ssdq.BF16, ssdq.E4M3, ssdq.FP32, ssdq.INT8, ssdq.INT4])
@pytest.mark.parametrize("rule", RULES)
@pytest.mark.parametrize("shape", SHAPES)
def test_edge_shapes_and_options(fmt, rule, shape):
    B, H, P, N, aps = shape
    if fmt == ssdq.FP32 and (N > 128 or rule != ssdq.RTN):
        pytest.skip("the FP32 twin never rounds and is built for N <= 128")
    rng = np.random.default_rng(hash((fmt, rule) + shape) % 2**32)
    f32 = np.float32
    A = -np.exp(rng.uniform(-4, 1, (H, N) if aps else (H,))).astype(f32)
    use_D = (B + H) % 2 == 0
    D = rng.normal(0, 0.1, H).astype(f32) if use_D else None
    wb = 16 if (P + N) % 3 else N
    sb = 0
    if oracle.has_block_scale(fmt):
        sb = 16 if P % 2 else N
    src = (rng.standard_normal((B * H * P, N)) * 0.3).astype(f32)
    base = 11
    if fmt == ssdq.FP32:
        h0 = (src.view(np.uint32).copy(), None)
    else:
        h0 = oracle.quantize_store(src, fmt, oracle.RTN, 1, scale_block=sb, weyl_block=wb)
    pair = Pair((B, H, P, N), fmt, rule, A, D, weyl_block=wb, scale_block=sb, layer=3, weyl_seed=2, sr_seed=12345,
                batch_index_base=base, h0_codes=h0[0], h0_scales=h0[1])
    for t in range(2, 6):
        x = rng.standard_normal((B, H, P)).astype(f32)
        dt = np.log1p(np.exp(rng.normal(-2, 1, (B, H)))).astype(f32)
        Bm = rng.standard_normal((B, N)).astype(f32)
        Cm = rng.standard_normal((B, N)).astype(f32)
        pair.step_gpu(t, x, dt, Bm, Cm)
        y_ref = pair.step_oracle(t, x, dt, Bm, Cm)
        pair.compare(t, x, dt, Bm, Cm, y_ref)


@pytest.mark.parametrize("fmt", [ssdq.FP16, ssdq.BF16, ssdq.E4M3, ssdq.INT8])
def test_extreme_values_saturate_and_keep_signed_zero(fmt):
    """Decay to (sub)normal dust, growth beyond the largest finite value, exact zeros of both signs."""
    rng = np.random.default_rng(5)
    B, H, P, N = 1, 4, 4, 128
    f32 = np.float32
    A = np.array([-40.0, -1e-6, -3.0, 0.0], f32)           # fast decay / almost none / medium / a = 1
    sb = N if oracle.has_block_scale(fmt) else 0
    for rule in RULES:
        pair = Pair((B, H, P, N), fmt, rule, A, None, weyl_block=N, scale_block=sb)
        for t in range(1, 40):
            big = (t % 7 == 3)
            x = (rng.standard_normal((B, H, P)) * (1e6 if big else 1.0)).astype(f32)
            if t % 5 == 0:
                x[:] = 0.0
            if t % 5 == 1:
                x[:] = -0.0
            dt = np.full((B, H), 2.0, f32)
            Bm = (rng.standard_normal((B, N)) * (1e3 if big else 1e-3)).astype(f32)
            Cm = rng.standard_normal((B, N)).astype(f32)
            h_old = oracle.dequantize(pair.state_h, pair.scales_h, fmt, sb).reshape(B, H, P, N).astype(np.float64)
            a = np.exp(np.maximum(2.0 * A.astype(np.float64), -87.0))[None, :, None, None]
            h_new = a * h_old + (2.0 * x.astype(np.float64))[..., None] * Bm.astype(np.float64)[:, None, None, :]
            absum = np.einsum("bhpn,bn->bhp", np.abs(h_new), np.abs(Cm.astype(np.float64)))
            pair.step_gpu(t, x, dt, Bm, Cm)
            y_ref = pair.step_oracle(t, x, dt, Bm, Cm)
            pair.compare(t, x, dt, Bm, Cm, y_ref, y_absum=absum)


def test_decode_driver_equals_repeated_updates_and_resumes():
    """ssd_decode_run over a ring of inputs == one ssd_state_update per (step, layer); and because every
    rule is a function of (index, t, seed) only, stopping and resuming reproduces the same bits."""
    cfg = workloads.CONFIGS[1].with_batch(3)
    L, T = 2, 12
    for rule in RULES:
        params = [workloads.layer_params(cfg, l, l) for l in range(L)]
        ins = [[workloads.step_inputs(cfg, t, l, l) for l in range(L)] for t in range(1, T + 1)]
        stack = lambda i: to_dev(np.stack([np.stack([ins[t][l][i] for l in range(L)]) for t in range(T)]))
        xs, dts, Bs, Cs = (stack(i) for i in range(4))
        ys = torch.zeros_like(xs)

        def fresh():
            states = [torch.zeros(cfg.state_shape, dtype=torch.int16, device="cuda") for _ in range(L)]
            descs = [ssdq.make_desc(states[l], None, cfg.fmt, A=to_dev(params[l][0]), D=to_dev(params[l][1]), rule=rule,
                                    weyl=ssdq.weyl_offsets_init(l, 0, cfg.weyl_block), sr_seed=l, layer=l) for l in range(L)]
            return states, descs

        s1, d1 = fresh()
        ssdq.ssd_decode_run(d1, 1, T, ssdq.make_step_inputs(xs, dts, Bs, Cs, ys))
        s2, d2 = fresh()
        y2 = torch.zeros_like(ys)
        for t in range(T):
            for l in range(L):
                ssdq.ssd_state_update(d2[l], t + 1, x=xs[t, l], dt=dts[t, l], Bm=Bs[t, l], Cm=Cs[t, l], y=y2[t, l])
        s3, d3 = fresh()
        y3 = torch.zeros_like(ys)
        ssdq.ssd_decode_run(d3, 1, 5, ssdq.make_step_inputs(xs[:5], dts[:5], Bs[:5], Cs[:5], y3[:5]))
        torch.cuda.synchronize()
        saved = [s.clone() for s in s3]                       # "checkpoint": the codes are the whole state
        s4, d4 = fresh()
        for l in range(L):
            s4[l].copy_(saved[l])
        ssdq.ssd_decode_run(d4, 6, T - 5, ssdq.make_step_inputs(xs[5:], dts[5:], Bs[5:], Cs[5:], y3[5:]))
        torch.cuda.synchronize()
        for l in range(L):
            assert torch.equal(s1[l], s2[l]) and torch.equal(s1[l], s4[l])
        assert torch.equal(ys, y2) and torch.equal(ys, y3)
        # and the oracle agrees on the final state
        for l in range(L):
            st, _ = oracle.new_state(cfg.state_shape, cfg.fmt)
            for t in range(T):
                oracle.state_update(st, None, cfg.fmt, 0, *ins[t][l][:2], params[l][0], *ins[t][l][2:], params[l][1], rule,
                                    t + 1, layer=l, weyl_block=cfg.weyl_block, sr_seed=l)
            assert np.array_equal(codes_to_host(s1[l], cfg.fmt), st)


def test_ring_reuses_inputs():
    cfg = workloads.CONFIGS[1]
    A, D = workloads.layer_params(cfg)
    ring, T = 3, 7
    ins = [workloads.step_inputs(cfg, t) for t in range(1, ring + 1)]
    stack = lambda i: to_dev(np.stack([ins[t][i][None] for t in range(ring)]))
    xs, dts, Bs, Cs = (stack(i) for i in range(4))
    ys = torch.zeros_like(xs)
    state = torch.zeros(cfg.state_shape, dtype=torch.int16, device="cuda")
    desc = ssdq.make_desc(state, None, cfg.fmt, A=to_dev(A), D=to_dev(D), rule=ssdq.WEYL, weyl=ssdq.weyl_offsets_init(0, 0, 16))
    ssdq.ssd_decode_run([desc], 1, T, ssdq.make_step_inputs(xs, dts, Bs, Cs, ys))
    st, _ = oracle.new_state(cfg.state_shape, cfg.fmt)
    for i in range(T):
        x, dt, Bm, Cm = ins[i % ring]
        oracle.state_update(st, None, cfg.fmt, 0, x, dt, A, Bm, Cm, D, oracle.WEYL, 1 + i, weyl_block=16)
    torch.cuda.synchronize()
    assert np.array_equal(codes_to_host(state, cfg.fmt), st)


@pytest.mark.parametrize("staging_slots,host_ring", [(2, 12), (3, 12), (2, 4)])
def test_host_buffer_driver_equals_device_driver(staging_slots, host_ring):
    """ssd_decode_run_host (pinned host inputs, y back to host, copies overlapped with compute) produces the
    bits of ssd_decode_run on device-resident inputs."""
    cfg = workloads.CONFIGS[1].with_batch(3)
    L, T = 2, 12
    params = [workloads.layer_params(cfg, l, l) for l in range(L)]
    ins = [[workloads.step_inputs(cfg, 1 + (t % host_ring), l, l) for l in range(L)] for t in range(T)]
    stack_h = lambda i: torch.from_numpy(np.stack([np.stack([ins[t][l][i] for l in range(L)]) for t in range(host_ring)])).pin_memory()
    xs_h, dts_h, Bs_h, Cs_h = (stack_h(i) for i in range(4))
    ys_h = torch.zeros_like(xs_h).pin_memory()

    def fresh():
        states = [torch.zeros(cfg.state_shape, dtype=torch.int16, device="cuda") for _ in range(L)]
        descs = [ssdq.make_desc(states[l], None, cfg.fmt, A=to_dev(params[l][0]), D=to_dev(params[l][1]), rule=ssdq.WEYL,
                                weyl=ssdq.weyl_offsets_init(l, 0, cfg.weyl_block), layer=l) for l in range(L)]
        return states, descs

    s1, d1 = fresh()
    xs, dts, Bs, Cs = (t.cuda() for t in (xs_h, dts_h, Bs_h, Cs_h))
    ys = torch.zeros_like(xs)
    ssdq.ssd_decode_run(d1, 1, T, ssdq.make_step_inputs(xs, dts, Bs, Cs, ys))
    s2, d2 = fresh()
    stg = [torch.zeros((staging_slots,) + tuple(t.shape[1:]), dtype=torch.float32, device="cuda") for t in (xs_h, dts_h, Bs_h, Cs_h, ys_h)]
    for _ in range(2):          # twice: the second call reuses the driver's streams and events
        for st in s2:
            st.zero_()
        ys_h.zero_()
        ssdq.ssd_decode_run_host(d2, 1, T, ssdq.make_step_inputs(xs_h, dts_h, Bs_h, Cs_h, ys_h), ssdq.make_step_inputs(*stg))
        torch.cuda.current_stream().synchronize()
        for l in range(L):
            assert torch.equal(s1[l], s2[l])
        assert torch.equal(ys.cpu(), ys_h)


@pytest.mark.parametrize("fmt", [ssdq.BF16, ssdq.FP16, ssdq.E4M3, ssdq.INT8])
@pytest.mark.parametrize("rule", [ssdq.RTN, ssdq.WEYL])
@pytest.mark.parametrize("shape,groups,aps", [((2, 8, 64, 128), 4, False), ((3, 6, 5, 64), 2, False), ((2, 12, 1, 16), 3, True)])
def test_production_signature_options(fmt, rule, shape, groups, aps):
    """dt_bias + in-kernel softplus, grouped B and C, z gate: state bit for bit, gated y to tolerance, on the tile
    kernel's shape and on generic ones."""
    B, H, P, N = shape
    rng = np.random.default_rng(hash((fmt, rule) + shape) % 2**32)
    f32 = np.float32
    A = -np.exp(rng.uniform(-4, 1, (H, N) if aps else (H,))).astype(f32)
    D = rng.normal(0, 0.1, H).astype(f32)
    bias = rng.normal(-2, 1, H).astype(f32)
    sb = N if oracle.has_block_scale(fmt) else 0
    pair = Pair(shape, fmt, rule, A, D, weyl_block=16, scale_block=sb, dt_bias=bias, dt_softplus=True, ngroups=groups)
    for t in range(1, 6):
        x = rng.standard_normal((B, H, P)).astype(f32)
        raw = rng.normal(-1, 2, (B, H)).astype(f32)
        raw[0, 0] = 25.0                                            # beyond the softplus threshold
        Bm = (rng.standard_normal((B, groups, N)) * 0.3).astype(f32)
        Cm = rng.standard_normal((B, groups, N)).astype(f32)
        z = rng.standard_normal((B, H, P)).astype(f32) * 2
        y = pair.step_gpu(t, x, raw, Bm, Cm, z).cpu().numpy()
        y_ref = pair.step_oracle(t, x, raw, Bm, Cm, z)
        torch.cuda.synchronize()
        assert np.array_equal(codes_to_host(pair.state_d, fmt), pair.state_h), t
        if pair.scales_h is not None:
            assert np.array_equal(pair.scales_d.cpu().numpy().view(np.uint32), pair.scales_h.view(np.uint32))
        # tolerance: the ungated bound times |silu(z)|, plus the gate's own relative error
        new_f32 = oracle.dequantize(pair.state_h, pair.scales_h, fmt, sb).reshape(shape).astype(np.float64)
        Cexp = np.repeat(Cm, H // groups, axis=1).astype(np.float64)            # [B, H, N]
        absum = np.einsum("bhpn,bhn->bhp", np.abs(new_f32), np.abs(Cexp)) + np.abs(D.astype(np.float64))[None, :, None] * np.abs(x)
        gate = np.abs(z.astype(np.float64) / (1 + np.exp(-z.astype(np.float64))))
        assert np.all(np.abs(y - y_ref) <= 1e-5 * absum * gate + 4e-6 * np.abs(y_ref) + 1e-30), t


@pytest.mark.parametrize("fmt", [ssdq.FP16, ssdq.BF16, ssdq.E4M3, ssdq.INT8])
@pytest.mark.parametrize("rule", RULES)
def test_replay_step_matches_oracle_and_the_decode_step(fmt, rule):
    """ssd_replay_step on recorded (a, w) traces: equal to the oracle's replay, and -- fed a = exp_spec(dt A) and
    w = (dt x) B from the host -- equal to the fused decode step's state."""
    rng = np.random.default_rng(70 + fmt)
    B, H, P, N = 3, 5, 8, 128
    f32 = np.float32
    sb = N if oracle.has_block_scale(fmt) else 0
    A = -np.exp(rng.uniform(-3, 1, H)).astype(f32)
    pair = Pair((B, H, P, N), fmt, rule, A, None, weyl_block=16, scale_block=sb, layer=2, sr_seed=5, batch_index_base=4)
    codes_h, scales_h = pair.state_h.reshape(-1, N).copy(), None if pair.scales_h is None else pair.scales_h.copy()
    codes_d, scales_d = codes_to_dev(codes_h, fmt), to_dev(scales_h)
    weyl = ssdq.weyl_offsets_init(2, 0, 16)
    base = 4 * H * P
    for t in range(1, 6):
        x = rng.standard_normal((B, H, P)).astype(f32)
        dt = np.log1p(np.exp(rng.normal(-2, 0.5, (B, H)))).astype(f32)
        Bm = rng.standard_normal((B, N)).astype(f32)
        Cm = rng.standard_normal((B, N)).astype(f32)
        pair.step_gpu(t, x, dt, Bm, Cm)
        a = oracle.exp_spec((dt * A[None, :]).astype(f32).ravel())
        w = ((dt[:, :, None] * x).astype(f32)[..., None] * Bm[:, None, None, :]).astype(f32).reshape(-1, N)
        ssdq.replay_step(to_dev(w), to_dev(a), P, codes_d, scales_d, fmt, rule, t, weyl=weyl, sr_seed=5, layer=2,
                         scale_block=sb, row_index_base=base)
        oracle.replay_step(w, a, P, codes_h, scales_h, fmt, rule, t, scale_block=sb, layer=2, weyl_block=16, sr_seed=5,
                           row_index_base=base)
        torch.cuda.synchronize()
        assert np.array_equal(codes_to_host(codes_d, fmt), codes_h), t
        assert np.array_equal(codes_to_host(pair.state_d, fmt).reshape(-1, N), codes_h), t
        if scales_h is not None:
            assert np.array_equal(scales_d.cpu().numpy().view(np.uint32), scales_h.view(np.uint32))


@pytest.mark.parametrize("fmt", [ssdq.BF16, ssdq.E4M3, ssdq.INT8])
@pytest.mark.parametrize("rule", [ssdq.RTN, ssdq.WEYL, ssdq.SR])
def test_checkpointed_rounding(fmt, rule):
    """Only every k-th write is rounded (CC = k).  k = 1 reproduces the plain driver; k = 4 equals the oracle's FP32
    update with a quantise / dequantise round trip at every fourth write."""
    from dataclasses import replace
    cfg = replace(workloads.CONFIGS[4], batch=2, nheads=4, fmt=fmt)
    sb, wb = cfg.scale_block if oracle.has_block_scale(fmt) else 0, cfg.weyl_block
    T = 12
    A, D = workloads.layer_params(cfg)
    ins = [workloads.step_inputs(cfg, t) for t in range(1, T + 1)]
    stack = lambda i: to_dev(np.stack([ins[t][i][None] for t in range(T)]))
    xs, dts, Bs, Cs = (stack(i) for i in range(4))

    def fresh():
        st_h, sc_h = oracle.new_state(cfg.state_shape, fmt, sb)
        st, sc = codes_to_dev(st_h, fmt), to_dev(sc_h)
        desc = ssdq.make_desc(st, sc, fmt, A=to_dev(A), D=to_dev(D), rule=rule, weyl=ssdq.weyl_offsets_init(0, 0, wb), sr_seed=1,
                              scale_block=sb)
        return st, sc, desc

    s1, c1, d1 = fresh()
    y1 = torch.zeros_like(xs)
    ssdq.ssd_decode_run([d1], 1, T, ssdq.make_step_inputs(xs, dts, Bs, Cs, y1))
    s2, c2, d2 = fresh()
    y2 = torch.zeros_like(xs)
    work = torch.zeros(cfg.state_shape, dtype=torch.float32, device="cuda")
    ssdq.ssd_decode_run_checkpointed([d2], [work], 1, 1, T, ssdq.make_step_inputs(xs, dts, Bs, Cs, y2))
    torch.cuda.synchronize()
    assert torch.equal(s1, s2) and (c1 is None or torch.equal(c1, c2))
    assert torch.allclose(y1, y2, rtol=0, atol=1e-5 * float(y1.abs().max()))
    # k = 4 against the oracle
    s3, c3, d3 = fresh()
    y3 = torch.zeros_like(xs)
    work.zero_()
    ssdq.ssd_decode_run_checkpointed([d3], [work], 4, 1, T, ssdq.make_step_inputs(xs, dts, Bs, Cs, y3))
    w_h = np.zeros(cfg.state_shape, np.uint32)
    N = cfg.dstate
    for t in range(1, T + 1):
        x, dt, Bm, Cm = ins[t - 1]
        oracle.state_update(w_h, None, oracle.FP32, 0, x, dt, A, Bm, Cm, D, oracle.RTN, t)
        if t % 4 == 0:
            codes, scales = oracle.quantize_store(w_h.view(np.float32).reshape(-1, N), fmt, rule, t, scale_block=sb, weyl_block=wb, sr_seed=1)
            w_h = oracle.dequantize(codes, scales, fmt, sb).reshape(cfg.state_shape).view(np.uint32).copy()
    torch.cuda.synchronize()
    assert np.array_equal(codes_to_host(s3, fmt).reshape(-1, N), codes)
    assert np.array_equal(work.cpu().numpy().view(np.uint32), w_h)


def test_drivers_carry_the_gate_and_the_options():
    """z, dt_bias, softplus and groups through ssd_decode_run and ssd_decode_run_host equal per-step calls."""
    from dataclasses import replace
    cfg = replace(workloads.CONFIGS[5], batch=2, nheads=4, n_layers=1)
    B, H, P, N = cfg.state_shape
    G, T = 2, 6
    rng = np.random.default_rng(17)
    f32 = np.float32
    A, D = workloads.layer_params(cfg)
    bias = rng.normal(-2, 0.5, H).astype(f32)
    xs_h = torch.from_numpy(rng.standard_normal((T, 1, B, H, P)).astype(f32)).pin_memory()
    dts_h = torch.from_numpy(rng.normal(-1, 1, (T, 1, B, H)).astype(f32)).pin_memory()
    Bs_h = torch.from_numpy((rng.standard_normal((T, 1, B, G, N)) * 0.2).astype(f32)).pin_memory()
    Cs_h = torch.from_numpy(rng.standard_normal((T, 1, B, G, N)).astype(f32)).pin_memory()
    zs_h = torch.from_numpy(rng.standard_normal((T, 1, B, H, P)).astype(f32)).pin_memory()
    xs, dts, Bs, Cs, zs = (t.cuda() for t in (xs_h, dts_h, Bs_h, Cs_h, zs_h))

    def fresh():
        st = torch.zeros(cfg.state_shape, dtype=torch.int16, device="cuda")
        return st, ssdq.make_desc(st, None, cfg.fmt, A=to_dev(A), D=to_dev(D), rule=ssdq.WEYL, weyl=ssdq.weyl_offsets_init(0, 0, N),
                                  dt_bias=to_dev(bias), dt_softplus=True, ngroups=G)

    s1, d1 = fresh()
    y1 = torch.zeros_like(xs)
    for t in range(T):
        ssdq.ssd_state_update(d1, t + 1, x=xs[t, 0], dt=dts[t, 0], Bm=Bs[t, 0], Cm=Cs[t, 0], y=y1[t, 0], z=zs[t, 0])
    s2, d2 = fresh()
    y2 = torch.zeros_like(xs)
    ssdq.ssd_decode_run([d2], 1, T, ssdq.make_step_inputs(xs, dts, Bs, Cs, y2, zs))
    s3, d3 = fresh()
    y3_h = torch.zeros_like(xs_h).pin_memory()
    stg = [torch.zeros((2,) + tuple(t.shape[1:]), dtype=torch.float32, device="cuda") for t in (xs_h, dts_h, Bs_h, Cs_h, y3_h, zs_h)]
    ssdq.ssd_decode_run_host([d3], 1, T, ssdq.make_step_inputs(xs_h, dts_h, Bs_h, Cs_h, y3_h, zs_h), ssdq.make_step_inputs(*stg))
    torch.cuda.synchronize()
    assert torch.equal(s1, s2) and torch.equal(s1, s3)
    assert torch.equal(y1, y2) and torch.equal(y1.cpu(), y3_h)
    # and the oracle agrees with the state
    st, _ = oracle.new_state(cfg.state_shape, cfg.fmt)
    for t in range(T):
        oracle.state_update(st, None, cfg.fmt, 0, xs_h[t, 0].numpy(), dts_h[t, 0].numpy(), A, Bs_h[t, 0].numpy(), Cs_h[t, 0].numpy(), D,
                            oracle.WEYL, t + 1, weyl_block=N, dt_bias=bias, dt_softplus=True, ngroups=G, z=zs_h[t, 0].numpy())
    assert np.array_equal(codes_to_host(s1, cfg.fmt), st)


@pytest.mark.parametrize("rule", RULES)
def test_graph_replay_equals_the_plain_driver(rule):
    """A captured graph of 4 steps x 2 layers, replayed three times with the write index kept in device memory,
    equals 12 steps of ssd_decode_run."""
    cfg = workloads.CONFIGS[1].with_batch(3)
    L, ring, spl, reps = 2, 2, 4, 3
    params = [workloads.layer_params(cfg, l, l) for l in range(L)]
    ins = [[workloads.step_inputs(cfg, t + 1, l, l) for l in range(L)] for t in range(ring)]
    stack = lambda i: to_dev(np.stack([np.stack([ins[t][l][i] for l in range(L)]) for t in range(ring)]))
    xs, dts, Bs, Cs = (stack(i) for i in range(4))

    def fresh():
        states = [torch.zeros(cfg.state_shape, dtype=torch.int16, device="cuda") for _ in range(L)]
        descs = [ssdq.make_desc(states[l], None, cfg.fmt, A=to_dev(params[l][0]), D=to_dev(params[l][1]), rule=rule,
                                weyl=ssdq.weyl_offsets_init(l, 0, cfg.weyl_block), sr_seed=l, layer=l) for l in range(L)]
        return states, descs

    s1, d1 = fresh()
    y1 = torch.zeros_like(xs)
    ssdq.ssd_decode_run(d1, 1, spl * reps, ssdq.make_step_inputs(xs, dts, Bs, Cs, y1))
    s2, d2 = fresh()
    y2 = torch.zeros_like(xs)
    counter = torch.zeros(1, dtype=torch.int32, device="cuda")
    graph = ssdq.DecodeGraph(d2, spl, ssdq.make_step_inputs(xs, dts, Bs, Cs, y2), counter)
    for _ in range(reps):
        graph.launch()
    torch.cuda.synchronize()
    assert int(counter.item()) == spl * reps
    for l in range(L):
        assert torch.equal(s1[l], s2[l])
    assert torch.equal(y1, y2)
    graph.close()


def test_graph_replay_on_the_persistent_kernel():
    """The replayable graph over the one-byte persistent kernel (whose one-time set-up must happen before the capture
    begins: this instantiation -- E4M3, hash SR, heads of 128 rows, one scale per 16 entries -- is launched nowhere else
    before): equal to the plain driver."""
    from dataclasses import replace
    cfg = replace(workloads.CONFIGS[4], batch=2, nheads=6, headdim=128, scale_block=16)
    L, ring, spl, reps = 2, 2, 2, 3
    rule = ssdq.SR_HASH
    params = [workloads.layer_params(cfg, l, l) for l in range(L)]
    ins = [[workloads.step_inputs(cfg, t + 1, l, l) for l in range(L)] for t in range(ring)]
    stack = lambda i: to_dev(np.stack([np.stack([ins[t][l][i] for l in range(L)]) for t in range(ring)]))
    xs, dts, Bs, Cs = (stack(i) for i in range(4))

    def fresh():
        states = [torch.zeros(cfg.state_shape, dtype=torch.uint8, device="cuda") for _ in range(L)]
        scales = [torch.full((cfg.entries_per_layer // 16,), float(np.finfo(np.float32).tiny), device="cuda") for _ in range(L)]
        descs = [ssdq.make_desc(states[l], scales[l], cfg.fmt, A=to_dev(params[l][0]), D=to_dev(params[l][1]), rule=rule,
                                weyl=ssdq.weyl_offsets_init(l, 0, cfg.weyl_block), sr_seed=l, layer=l, scale_block=16) for l in range(L)]
        return states, scales, descs

    s2, c2, d2 = fresh()
    y2 = torch.zeros_like(xs)
    counter = torch.zeros(1, dtype=torch.int32, device="cuda")
    graph = ssdq.DecodeGraph(d2, spl, ssdq.make_step_inputs(xs, dts, Bs, Cs, y2), counter)     # first use of the instantiation
    for _ in range(reps):
        graph.launch()
    torch.cuda.synchronize()
    assert ssdq.last_kernel() == "ssd_update_stream_kernel"
    s1, c1, d1 = fresh()
    y1 = torch.zeros_like(xs)
    ssdq.ssd_decode_run(d1, 1, spl * reps, ssdq.make_step_inputs(xs, dts, Bs, Cs, y1))
    torch.cuda.synchronize()
    for l in range(L):
        assert torch.equal(s1[l], s2[l]) and torch.equal(c1[l], c2[l])
    assert torch.equal(y1, y2)
    graph.close()


HEAD_SHARD_CASES = [
    # fmt, (B, H_global, P, N), per-state A, scale granularity, kernel family the shard runs on
    (ssdq.BF16, (3, 6, 64, 128), False, None, "ssd_update_tile_kernel"),
    (ssdq.FP16, (3, 6, 64, 64), False, None, "ssd_update_tile_kernel"),
    (ssdq.E4M3, (3, 6, 64, 128), False, "row", "ssd_update_stream_kernel"),
    (ssdq.INT8, (3, 6, 128, 128), False, "block16", "ssd_update_stream_kernel"),
    (ssdq.E4M3, (3, 6, 64, 128), False, "head", "ssd_update_headscale_kernel"),
    (ssdq.BF16, (5, 96, 1, 16), True, None, "ssd_update_mamba1_kernel"),
    (ssdq.INT8, (5, 96, 1, 16), True, "row", "ssd_update_mamba1_kernel"),
    (ssdq.BF16, (3, 6, 8, 32), True, None, "ssd_update_kernel"),
]


@pytest.mark.parametrize("rule", [ssdq.WEYL, ssdq.SR, ssdq.SR_HASH])
@pytest.mark.parametrize("fmt,shape,aps,scale,family", HEAD_SHARD_CASES)
def test_a_head_shard_reproduces_the_bits_of_the_whole_layer(fmt, shape, aps, scale, family, rule):
    """Tensor-parallel split: a call that holds heads [h0, h1) of the layer, told head_index_base = h0 and
    nheads_global = H, writes the codes that the unsharded call writes for those heads (the thresholds of Eq. 2 are
    drawn at the entry's index in the whole layer: Appendix B "Dithers" numbers the rows of the full state matrix).
    Checked against the oracle on the shard and against the library's own unsharded run, with a batch offset on top."""
    B, Hg, P, N = shape
    f32 = np.float32
    rng = np.random.default_rng(hash((fmt, shape, aps)) % 2**31)
    sb = {None: 0, "row": N, "block16": 16, "head": P * N}[scale]
    A = (-np.exp(rng.uniform(-3, 1, (Hg, N) if aps else Hg))).astype(f32)
    D = rng.normal(0, 0.1, Hg).astype(f32)
    wb = 16
    bbase = 7
    whole = Pair((B, Hg, P, N), fmt, rule, A, D, weyl_block=wb, scale_block=sb, layer=3, weyl_seed=2, sr_seed=11, batch_index_base=bbase)
    h0 = Hg // 3
    h1 = Hg - Hg // 6
    part = Pair((B, h1 - h0, P, N), fmt, rule, A[h0:h1].copy(), D[h0:h1].copy(), weyl_block=wb, scale_block=sb, layer=3, weyl_seed=2,
                sr_seed=11, batch_index_base=bbase, head_index_base=h0, nheads_global=Hg)
    for t in range(1, 5):
        x = rng.standard_normal((B, Hg, P)).astype(f32)
        dt = np.log1p(np.exp(rng.normal(-2, 0.5, (B, Hg)))).astype(f32)
        Bm = (rng.standard_normal((B, N)) / np.sqrt(N)).astype(f32)
        Cm = rng.standard_normal((B, N)).astype(f32)
        whole.step_gpu(t, x, dt, Bm, Cm)
        xs, dts = np.ascontiguousarray(x[:, h0:h1]), np.ascontiguousarray(dt[:, h0:h1])
        part.step_gpu(t, xs, dts, Bm, Cm)
        assert ssdq.last_kernel() == family
        y_ref = part.step_oracle(t, xs, dts, Bm, Cm)
        part.compare(t, xs, dts, Bm, Cm, y_ref)
        assert np.array_equal(codes_to_host(part.state_d, fmt), codes_to_host(whole.state_d, fmt)[:, h0:h1]), t
        if part.scales_d is not None:
            ws = whole.scales_d.cpu().numpy().reshape(B, Hg, -1)[:, h0:h1]
            assert np.array_equal(part.scales_d.cpu().numpy().reshape(B, h1 - h0, -1), ws), t
        assert np.array_equal(part.y_d.cpu().numpy(), whole.y_d.cpu().numpy()[:, h0:h1]), t


def test_head_shard_arguments_are_checked():
    st = torch.zeros((2, 4, 16, 64), dtype=torch.int16, device="cuda")
    A = torch.zeros(4, device="cuda")
    x = torch.zeros((2, 4, 16), device="cuda"); dt = torch.zeros((2, 4), device="cuda"); Bm = torch.zeros((2, 64), device="cuda")
    for hb, hg in ((1, 0), (1, 4), (0, 3), (5, 8)):
        d = ssdq.make_desc(st, None, ssdq.BF16, A=A, D=None, rule=ssdq.RTN, head_index_base=hb, nheads_global=hg)
        with pytest.raises(ssdq.SsdqError) as e:
            ssdq.ssd_state_update(d, 1, x=x, dt=dt, Bm=Bm, Cm=Bm, y=torch.empty_like(x))
        assert e.value.status == ssdq.ERR_SHAPE
    d = ssdq.make_desc(st, None, ssdq.BF16, A=A, D=None, rule=ssdq.RTN, head_index_base=4, nheads_global=8)
    ssdq.ssd_state_update(d, 1, x=x, dt=dt, Bm=Bm, Cm=Bm, y=torch.empty_like(x))


@pytest.mark.parametrize("fmt", [ssdq.BF16, ssdq.INT8])
@pytest.mark.parametrize("rule", [ssdq.WEYL, ssdq.SR])
def test_checkpointed_rounding_on_a_head_shard(fmt, rule):
    """The checkpointing driver rounds a head shard's rows at their indices in the whole layer: heads 1..2 of 4, every
    second write rounded, equal the same heads of the unsharded checkpointed run."""
    from dataclasses import replace
    cfg = replace(workloads.CONFIGS[4], batch=3, nheads=4, fmt=fmt)
    sb, wb = (cfg.scale_block if oracle.has_block_scale(fmt) else 0), cfg.weyl_block
    T, h0, h1 = 6, 1, 3
    A, D = workloads.layer_params(cfg)
    ins = [workloads.step_inputs(cfg, t) for t in range(1, T + 1)]
    stack = lambda i, sl: to_dev(np.stack([np.ascontiguousarray(ins[t][i][:, sl] if i < 2 else ins[t][i])[None] for t in range(T)]))

    def run(sl, **shard):
        nh = len(range(*sl.indices(cfg.nheads)))
        shape = (cfg.batch, nh) + cfg.state_shape[2:]
        st_h, sc_h = oracle.new_state(shape, fmt, sb)
        st, sc = codes_to_dev(st_h, fmt), to_dev(sc_h)
        desc = ssdq.make_desc(st, sc, fmt, A=to_dev(A[sl].copy()), D=to_dev(D[sl].copy()), rule=rule,
                              weyl=ssdq.weyl_offsets_init(0, 0, wb), sr_seed=1, scale_block=sb, batch_index_base=5, **shard)
        xs, dts, Bs, Cs = (stack(i, sl) for i in range(4))
        y = torch.zeros_like(xs)
        work = torch.zeros(shape, dtype=torch.float32, device="cuda")
        ssdq.ssd_decode_run_checkpointed([desc], [work], 2, 1, T, ssdq.make_step_inputs(xs, dts, Bs, Cs, y))
        torch.cuda.synchronize()
        return st, sc, y

    st_w, sc_w, y_w = run(slice(0, cfg.nheads))
    st_p, sc_p, y_p = run(slice(h0, h1), head_index_base=h0, nheads_global=cfg.nheads)
    assert torch.equal(st_p, st_w[:, h0:h1])
    if sc_w is not None:
        assert torch.equal(sc_p.reshape(cfg.batch, h1 - h0, -1), sc_w.reshape(cfg.batch, cfg.nheads, -1)[:, h0:h1])
    assert torch.equal(y_p, y_w[:, :, :, h0:h1])


@pytest.mark.parametrize("fmt,shape,sb", [(ssdq.BF16, (2, 8, 64, 128), 0), (ssdq.E4M3, (2, 8, 64, 128), 128),
                                           (ssdq.INT8, (2, 8, 64, 128), 64 * 128), (ssdq.BF16, (3, 256, 1, 16), 0),
                                           (ssdq.FP16, (2, 3, 8, 32), 0),
                                           (ssdq.BF16, (16, 64, 64, 128), 0)])      # 1024 CTAs: the many-wave order of the gate
@pytest.mark.parametrize("L", [1, 3])       # one layer: every launch reads what the launch just before it wrote
def test_launch_overlap_does_not_change_a_bit(fmt, shape, sb, L):
    """The drivers launch their kernels with programmatic dependent launch by default (a kernel is scheduled while the one
    before it drains and waits for it before touching memory).  Three layers, 24 steps through ssd_decode_run and through
    a replayed graph, with the setting on and off: the same codes, scales and y, and the oracle's codes after the run."""
    B, H, P, N = shape
    f32 = np.float32
    T = 24 if L == 3 else 48
    rng = np.random.default_rng(5 + fmt)
    aps = (P == 1)
    A = [(-np.exp(rng.uniform(-3, 1, (H, N) if aps else H))).astype(f32) for _ in range(L)]
    D = [rng.normal(0, 0.1, H).astype(f32) for _ in range(L)]
    xs_h = rng.standard_normal((T, L, B, H, P)).astype(f32)
    dts_h = np.log1p(np.exp(rng.normal(-2, 0.5, (T, L, B, H)))).astype(f32)
    Bs_h = (rng.standard_normal((T, L, B, N)) / np.sqrt(N)).astype(f32)
    Cs_h = rng.standard_normal((T, L, B, N)).astype(f32)
    xs, dts, Bs, Cs = (to_dev(a) for a in (xs_h, dts_h, Bs_h, Cs_h))

    def fresh():
        out = []
        for l in range(L):
            st_h, sc_h = oracle.new_state(shape, fmt, sb)
            st, sc = codes_to_dev(st_h, fmt), to_dev(sc_h)
            out.append((st, sc, ssdq.make_desc(st, sc, fmt, A=to_dev(A[l]), D=to_dev(D[l]), rule=ssdq.WEYL,
                                               weyl=ssdq.weyl_offsets_init(l, 0, 16), layer=l, scale_block=sb)))
        return out

    def run(overlap, graph):
        prev = ssdq.set_launch_overlap(overlap)
        try:
            layers = fresh()
            y = torch.zeros_like(xs)
            sin = ssdq.make_step_inputs(xs, dts, Bs, Cs, y)
            descs = [d for _, _, d in layers]
            if graph:
                counter = torch.zeros(1, dtype=torch.int32, device="cuda")
                g = ssdq.DecodeGraph(descs, T // 2, ssdq.make_step_inputs(xs[:T // 2], dts[:T // 2], Bs[:T // 2], Cs[:T // 2], y[:T // 2]), counter)
                g.launch()
                g.launch()
                torch.cuda.synchronize()
                g.close()
            else:
                ssdq.ssd_decode_run(descs, 1, T, sin)
                torch.cuda.synchronize()
            return layers, y
        finally:
            ssdq.set_launch_overlap(prev)

    assert ssdq.set_launch_overlap(True) is True           # on by default
    base = None
    for graph in (True, False):         # the graph replays the first half of the inputs twice: compared with itself only
        base, y0 = run(False, graph)
        got, y = run(True, graph)
        for (s0, c0, _), (s1, c1, _) in zip(base, got):
            assert torch.equal(s0, s1) and (c0 is None or torch.equal(c0, c1)), graph
        assert torch.equal(y0, y), graph
    # and the run is the oracle's (first layer)
    st_h, sc_h = oracle.new_state(shape, fmt, sb)
    for t in range(1, T + 1):
        oracle.state_update(st_h, sc_h, fmt, sb, xs_h[t - 1, 0], dts_h[t - 1, 0], A[0], Bs_h[t - 1, 0], Cs_h[t - 1, 0], D[0],
                            oracle.WEYL, t, layer=0, weyl_block=16)
    assert np.array_equal(codes_to_host(base[0][0], fmt), st_h)


@pytest.mark.parametrize("cfg_index,batch,fmt", [(4, 0, None), (5, 32, None), (5, 32, ssdq.INT8), (2, 512, None), (3, 0, None)])
def test_launch_overlap_at_full_size_on_one_layer(cfg_index, batch, fmt):
    """Full-size launches of one layer back to back (every kernel reads the state, and for the scaled stores the scales,
    that the kernel just before it wrote, on whichever SM it lands): 16 steps through ssd_decode_run with the
    programmatic-launch setting on and off end in the same codes, scales and y."""
    from dataclasses import replace
    cfg = replace(workloads.CONFIGS[cfg_index], n_layers=1)
    if batch:
        cfg = cfg.with_batch(batch)
    if fmt is not None:
        cfg = replace(cfg, fmt=fmt, scale_block=cfg.dstate)
    T = 16
    A, D = workloads.layer_params(cfg)
    ins = [workloads.step_inputs(cfg, t) for t in range(1, T + 1)]
    stack = lambda i: to_dev(np.stack([ins[t][i][None] for t in range(T)]))
    xs, dts, Bs, Cs = (stack(i) for i in range(4))
    sb = cfg.scale_block if oracle.has_block_scale(cfg.fmt) else 0

    def run(overlap):
        prev = ssdq.set_launch_overlap(overlap)
        try:
            st_h, sc_h = oracle.new_state(cfg.state_shape, cfg.fmt, sb)
            st, sc = codes_to_dev(st_h, cfg.fmt), to_dev(sc_h)
            desc = ssdq.make_desc(st, sc, cfg.fmt, A=to_dev(A), D=to_dev(D), rule=ssdq.WEYL,
                                  weyl=ssdq.weyl_offsets_init(0, 0, cfg.weyl_block), scale_block=sb)
            y = torch.zeros_like(xs)
            ssdq.ssd_decode_run([desc], 1, T, ssdq.make_step_inputs(xs, dts, Bs, Cs, y))
            torch.cuda.synchronize()
            return st, sc, y
        finally:
            ssdq.set_launch_overlap(prev)

    s0, c0, y0 = run(False)
    for _ in range(3):
        s1, c1, y1 = run(True)
        assert torch.equal(s0, s1) and (c0 is None or torch.equal(c0, c1)) and torch.equal(y0, y1)

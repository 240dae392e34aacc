"""Helpers shared by the GPU parity tests: run the same seeded inputs through the CUDA library
(via its C ABI) and through the CPU oracle, and compare."""
import numpy as np
import torch

import oracle
from paper_2609_39185_b200 import ssdq, workloads

TORCH_CODE = {ssdq.FP16: torch.int16, ssdq.BF16: torch.int16, ssdq.E4M3: torch.uint8, ssdq.FP32: torch.int32,
              ssdq.INT8: torch.uint8, ssdq.INT7: torch.uint8, ssdq.INT6: torch.uint8, ssdq.INT4: torch.uint8}
NP_VIEW = {ssdq.FP16: np.int16, ssdq.BF16: np.int16, ssdq.E4M3: np.uint8, ssdq.FP32: np.int32,
           ssdq.INT8: np.uint8, ssdq.INT7: np.uint8, ssdq.INT6: np.uint8, ssdq.INT4: np.uint8}


def to_dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


def codes_to_dev(codes, fmt):
    return torch.from_numpy(np.ascontiguousarray(codes).view(NP_VIEW[fmt])).cuda()


def codes_to_host(t, fmt):
    return t.cpu().numpy().view(oracle.CODE_DTYPE[fmt])


def y_close(y_gpu, y_ref, Cm, new_state_f32, D, x, rel=1e-5):
    """The readout tolerance: |dy| <= rel * (sum_n |C_n h'_n| + |D x|) per element (the FP32 summation
    order is free) and ||dy||_2 <= rel * ||y||_2 per step."""
    absum = np.einsum("bhpn,bn->bhp", np.abs(new_state_f32.astype(np.float64)), np.abs(Cm.astype(np.float64)))
    if D is not None:
        absum = absum + np.abs(D.astype(np.float64))[None, :, None] * np.abs(x.astype(np.float64))
    dy = np.abs(y_gpu.astype(np.float64) - y_ref.astype(np.float64))
    elem_ok = np.all(dy <= rel * absum + 1e-30)
    norm_ok = np.linalg.norm(dy) <= rel * np.linalg.norm(y_ref.astype(np.float64)) + 1e-30
    return bool(elem_ok and norm_ok), float(np.max(dy / (absum + 1e-30)))


class Pair:
    """One layer's state held twice: on the GPU (library) and on the host (oracle)."""

    def __init__(self, shape, fmt, rule, A, D, *, weyl_block=16, scale_block=0, layer=0, weyl_seed=0, sr_seed=0,
                 batch_index_base=0, h0_codes=None, h0_scales=None, dt_bias=None, dt_softplus=False, ngroups=1,
                 head_index_base=0, nheads_global=0):
        self.shape, self.fmt, self.rule = shape, fmt, rule
        self.A, self.D = A, D
        self.kw = dict(layer=layer, weyl_seed=weyl_seed, weyl_block=weyl_block, sr_seed=sr_seed,
                       batch_index_base=batch_index_base, dt_bias=dt_bias, dt_softplus=dt_softplus, ngroups=ngroups,
                       head_index_base=head_index_base, nheads_global=nheads_global)
        self.bias_d = to_dev(dt_bias)
        self.scale_block = scale_block
        if h0_codes is None:
            self.state_h, self.scales_h = oracle.new_state(shape, fmt, scale_block)
        else:
            self.state_h = h0_codes.reshape(shape).copy()
            self.scales_h = None if h0_scales is None else h0_scales.reshape(-1).copy()
        self.state_d = codes_to_dev(self.state_h, fmt)
        self.scales_d = to_dev(self.scales_h)
        self.A_d, self.D_d = to_dev(A), to_dev(D)
        weyl = ssdq.weyl_offsets_init(layer, weyl_seed, weyl_block)
        self.desc = ssdq.make_desc(self.state_d, self.scales_d, fmt, A=self.A_d, D=self.D_d, rule=rule, weyl=weyl,
                                   sr_seed=sr_seed, layer=layer, scale_block=scale_block,
                                   batch_index_base=batch_index_base, dt_bias=self.bias_d, dt_softplus=dt_softplus,
                                   ngroups=ngroups, head_index_base=head_index_base, nheads_global=nheads_global)
        self.y_d = torch.empty(shape[:3], dtype=torch.float32, device="cuda")

    def step_gpu(self, t, x, dt, Bm, Cm, z=None):
        self._ins = [to_dev(v) for v in (x, dt, Bm, Cm, z)]
        ssdq.ssd_state_update(self.desc, t, x=self._ins[0], dt=self._ins[1], Bm=self._ins[2], Cm=self._ins[3], y=self.y_d,
                              z=self._ins[4])
        return self.y_d

    def step_oracle(self, t, x, dt, Bm, Cm, z=None):
        return oracle.state_update(self.state_h, self.scales_h, self.fmt, self.scale_block, x, dt, self.A, Bm, Cm,
                                   self.D, self.rule, t, z=z, **self.kw)

    def compare(self, t, x, dt, Bm, Cm, y_ref, y_absum=None):
        torch.cuda.synchronize()
        got = codes_to_host(self.state_d, self.fmt)
        assert np.array_equal(got, self.state_h), self._diff_report(got, t)
        if self.scales_h is not None:
            assert np.array_equal(self.scales_d.cpu().numpy().view(np.uint32), self.scales_h.view(np.uint32)), f"scales differ at step {t}"
        if y_absum is not None:
            # steps on which h' leaves the format's range: the stored (saturated) state no longer gives the
            # scale of the unrounded h', so the caller supplies sum_n |C_n h'_n| + |D x| itself
            dy = np.abs(self.y_d.cpu().numpy().astype(np.float64) - y_ref.astype(np.float64))
            assert np.all(dy <= 1e-5 * y_absum + 1e-30), f"y differs at step {t}: {np.max(dy / (y_absum + 1e-30)):.3e}"
            return
        new_f32 = oracle.dequantize(self.state_h, self.scales_h, self.fmt, self.scale_block).reshape(self.shape)
        ok, worst = y_close(self.y_d.cpu().numpy(), y_ref, Cm, new_f32, self.D, x)
        assert ok, f"y outside tolerance at step {t}: worst ratio {worst:.3e}"

    def _diff_report(self, got, t):
        bad = np.argwhere(got != self.state_h)
        i = tuple(bad[0])
        return (f"state differs at step {t}: {len(bad)} of {got.size} codes; first at {i}: "
                f"gpu {int(got[i]):#x} oracle {int(self.state_h[i]):#x}")


def run_parity(cfg, rule, steps, *, layer=0, seed=0, batch_slice=None, batch_index_base=0, sr_seed=0, weyl_seed=0,
               check_every=1, h0=None):
    """Decode `steps` steps of one layer of `cfg` on both sides and compare after every `check_every` steps."""
    A, D = workloads.layer_params(cfg, layer, seed)
    shape = cfg.state_shape
    if batch_slice is not None:
        nb = len(range(*batch_slice.indices(cfg.batch)))
        shape = (nb,) + shape[1:]
    pair = Pair(shape, cfg.fmt, rule, A, D, weyl_block=cfg.weyl_block, scale_block=cfg.scale_block, layer=layer,
                weyl_seed=weyl_seed, sr_seed=sr_seed, batch_index_base=batch_index_base,
                h0_codes=None if h0 is None else h0[0], h0_scales=None if h0 is None else h0[1])
    for t in range(1, steps + 1):
        ins = workloads.step_inputs(cfg, t, layer, seed, batch_slice)
        pair.step_gpu(t, *ins)
        y_ref = pair.step_oracle(t, *ins)
        if t % check_every == 0 or t == steps:
            pair.compare(t, *ins, y_ref)
    return pair

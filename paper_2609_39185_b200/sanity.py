"""Sanity report of the rule ordering: decode a workload with RTN, SR and the Weyl dither next to a
full-precision (FP32-state) twin on the same inputs, all on the GPU through the library, and log the
open-loop state error sum (h_hat - h)^2 / sum h^2 (Appendix B "Open-loop replay"), split by head memory
bin tau = 1 / (1 - a_bar) (Appendix B "Memory bins"), and a surrogate readout KL (softmax over each
sequence's readout vector; the paper's KL is over a vocabulary that does not exist here).

    python -m paper_2609_39185_b200.sanity --config 4 --steps 4096 --log-every 256 --out report.jsonl

This is a check of ordering (RTN's error keeps growing on long-memory heads, the dithers level off),
not a parity test and not a reproduction of the paper's numbers, which need trained models.
"""
from __future__ import annotations

import argparse
import json
from dataclasses import replace

import numpy as np

from . import workloads

BINS = ((0.0, 10.0, "tau<10"), (10.0, 100.0, "tau10-100"), (100.0, 1000.0, "tau100-1000"), (1000.0, np.inf, "tau>=1000"))
RULES = (("rtn", 0), ("sr", 1), ("weyl", 2), ("sr_hash", 3))


def head_time_constants(cfg, A, mean_dt):
    """tau = 1 / (1 - exp(A * mean dt)) per head (mean over states for a per-state A)."""
    a_bar = np.exp(A.astype(np.float64) * mean_dt[:, None] if A.ndim == 2 else A.astype(np.float64) * mean_dt)
    if a_bar.ndim == 2:
        a_bar = a_bar.mean(axis=1)
    return 1.0 / np.maximum(1.0 - a_bar, 1e-12)


def run(cfg, steps, log_every, chunk=128, seed=0, layer=0, emit=print):
    import torch
    from . import ssdq
    A, D = workloads.layer_params(cfg, layer, seed)
    A_d, D_d = torch.from_numpy(A).cuda(), torch.from_numpy(D).cuda()
    code_dtype = torch.uint8 if workloads.CODE_BYTES[cfg.fmt] == 1 else torch.int16
    runs = {}
    for name, rid in RULES:
        st = torch.zeros(cfg.state_shape, dtype=code_dtype, device="cuda")
        sc = None
        if cfg.fmt in workloads.SCALED_FORMATS:
            sc = torch.full((cfg.entries_per_layer // cfg.scale_block,), float(np.finfo(np.float32).tiny),
                            dtype=torch.float32, device="cuda")
        desc = ssdq.make_desc(st, sc, cfg.fmt, A=A_d, D=D_d, rule=rid, weyl=ssdq.weyl_offsets_init(layer, 0, cfg.weyl_block),
                              sr_seed=seed, layer=layer, scale_block=cfg.scale_block)
        runs[name] = (st, sc, desc)
    twin = torch.zeros(cfg.state_shape, dtype=torch.float32, device="cuda")
    twin_desc = ssdq.make_desc(twin, None, ssdq.FP32, A=A_d, D=D_d, rule=ssdq.RTN, layer=layer)
    workspace = torch.empty(int(ssdq.lib().ssdq_state_error_workspace_bytes(cfg.batch, cfg.nheads)), dtype=torch.uint8, device="cuda")
    dt_sum = np.zeros(cfg.nheads)
    records = []
    t = 0
    while t < steps:
        n = min(chunk, steps - t)
        ins = [workloads.step_inputs(cfg, t + 1 + i, layer, seed) for i in range(n)]
        dt_sum += sum(i[1].astype(np.float64).mean(axis=0) for i in ins)
        stack = lambda k: torch.from_numpy(np.stack([i[k][None] for i in ins])).cuda()
        xs, dts, Bs, Cs = (stack(k) for k in range(4))
        ys = {name: torch.empty_like(xs) for name in list(runs) + ["twin"]}
        for name, (st, sc, desc) in runs.items():
            ssdq.ssd_decode_run([desc], t + 1, n, ssdq.make_step_inputs(xs, dts, Bs, Cs, ys[name]))
        ssdq.ssd_decode_run([twin_desc], t + 1, n, ssdq.make_step_inputs(xs, dts, Bs, Cs, ys["twin"]))
        t += n
        if t % log_every == 0 or t == steps:
            tau = head_time_constants(cfg, A, dt_sum / t)
            rec = {"step": t, "config": cfg.name, "format": workloads.FORMAT_NAMES[cfg.fmt]}
            for name, (st, sc, desc) in runs.items():
                e2, r2 = ssdq.state_error(st, sc, twin, cfg.fmt, cfg.scale_block, workspace)
                e2, r2 = e2.cpu().numpy(), r2.cpu().numpy()
                kl = ssdq.readout_kl(ys["twin"][n - 1, 0], ys[name][n - 1, 0]).cpu().numpy()
                entry = {"state_error": float(e2.sum() / max(r2.sum(), 1e-300)), "readout_kl": float(kl.mean())}
                for lo, hi, label in BINS:
                    m = (tau >= lo) & (tau < hi)
                    if m.any():
                        entry[label] = float(e2[m].sum() / max(r2[m].sum(), 1e-300))
                rec[name] = entry
            rec["heads_per_bin"] = {label: int(((tau >= lo) & (tau < hi)).sum()) for lo, hi, label in BINS}
            records.append(rec)
            emit(json.dumps(rec))
    return records


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--steps", type=int, default=0)
    ap.add_argument("--log-every", type=int, default=256)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--format", default="", choices=["", "fp16", "bf16", "e4m3", "int8", "int7", "int6", "int4"])
    ap.add_argument("--scale", default="", choices=["", "row", "block16", "head"], help="granularity of the FP32 scale of a scaled store")
    ap.add_argument("--out", default="")
    args = ap.parse_args()
    cfg = workloads.CONFIGS[args.config]
    if args.batch:
        cfg = cfg.with_batch(args.batch)
    cfg = replace(cfg, n_layers=1)
    if args.format:
        fmt = {v: k for k, v in workloads.FORMAT_NAMES.items()}[args.format]
        cfg = replace(cfg, fmt=fmt, scale_block=(cfg.scale_block or cfg.weyl_block) if fmt in workloads.SCALED_FORMATS else 0)
    if args.scale and cfg.fmt in workloads.SCALED_FORMATS:
        cfg = replace(cfg, scale_block={"row": cfg.dstate, "block16": 16, "head": cfg.headdim * cfg.dstate}[args.scale])
    out = open(args.out, "w") if args.out else None

    def emit(line):
        print(line)
        if out:
            out.write(line + "\n")

    run(cfg, args.steps or cfg.steps, args.log_every, emit=emit)


if __name__ == "__main__":
    main()

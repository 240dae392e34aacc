"""The N > 1 mode on CPU: two gloo ranks each run the oracle on their batch shard with the shard's
global batch base, then on their head shard with its head base; either way they reproduce the unsharded
run bit for bit together, and timings reduce by max."""
import os
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import oracle
    from paper_2609_39185_b200 import workloads
    from paper_2609_39185_b200.replicas import max_over_ranks, shard_batch_base
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    per_rank = 2
    cfg = workloads.CONFIGS[1].with_batch(per_rank * world)
    A, D = workloads.layer_params(cfg)
    base = shard_batch_base(rank, per_rank)
    sl = slice(base, base + per_rank)
    results = {}
    for rule in (oracle.SR, oracle.WEYL):
        st, _ = oracle.new_state((per_rank,) + cfg.state_shape[1:], cfg.fmt)
        for t in range(1, 9):
            x, dt, Bm, Cm = workloads.step_inputs(cfg, t, batch_slice=sl)
            oracle.state_update(st, None, cfg.fmt, 0, x, dt, A, Bm, Cm, D, rule, t, batch_index_base=base)
        results[rule] = st
    # the same layer split over the heads instead (tensor parallel): every sequence, this rank's heads
    from paper_2609_39185_b200.replicas import shard_head_range
    h0, h1 = shard_head_range(rank, world, cfg.nheads)
    heads = {}
    for rule in (oracle.SR, oracle.WEYL):
        st, _ = oracle.new_state((cfg.batch, h1 - h0) + cfg.state_shape[2:], cfg.fmt)
        for t in range(1, 9):
            x, dt, Bm, Cm = workloads.step_inputs(cfg, t)
            oracle.state_update(st, None, cfg.fmt, 0, np.ascontiguousarray(x[:, h0:h1]), np.ascontiguousarray(dt[:, h0:h1]),
                                A[h0:h1].copy(), Bm, Cm, D[h0:h1].copy(), rule, t, head_index_base=h0, nheads_global=cfg.nheads)
        heads[rule] = st
    slowest = max_over_ranks(1.0 + rank, dist)
    np.savez(os.path.join(out, f"rank{rank}.npz"), sr=results[oracle.SR], weyl=results[oracle.WEYL], slowest=slowest,
             sr_heads=heads[oracle.SR], weyl_heads=heads[oracle.WEYL])
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_equal_one_big_batch(tmp_path):
    world = 2
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    import oracle
    from paper_2609_39185_b200 import workloads
    cfg = workloads.CONFIGS[1].with_batch(4)
    A, D = workloads.layer_params(cfg)
    for name, rule in (("sr", oracle.SR), ("weyl", oracle.WEYL)):
        full, _ = oracle.new_state(cfg.state_shape, cfg.fmt)
        for t in range(1, 9):
            x, dt, Bm, Cm = workloads.step_inputs(cfg, t)
            oracle.state_update(full, None, cfg.fmt, 0, x, dt, A, Bm, Cm, D, rule, t)
        parts = [np.load(os.path.join(tmp_path, f"rank{r}.npz")) for r in range(world)]
        assert np.array_equal(np.concatenate([p[name] for p in parts]), full)
        assert np.array_equal(np.concatenate([p[name + "_heads"] for p in parts], axis=1), full)
        assert all(float(p["slowest"]) == 2.0 for p in parts)


def test_head_ranges_tile_the_layer():
    import pytest
    from paper_2609_39185_b200.replicas import shard_head_range
    assert [shard_head_range(r, 4, 128) for r in range(4)] == [(0, 32), (32, 64), (64, 96), (96, 128)]
    with pytest.raises(ValueError):
        shard_head_range(0, 3, 128)

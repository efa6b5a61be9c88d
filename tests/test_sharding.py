"""Host logic of runs on several GPUs, exercised with two CPU ranks over gloo.

The operator has no data-path collective (independent (batch, head) problems); what is tested is the
bookkeeping: distinct per-rank batches, disjoint covering batch slices, max-over-ranks time and summed
unit counts, and that the shards of a batch give exactly the rows of the unsharded oracle result.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2606_08804_b200 import inputs as gen
from paper_2606_08804_b200 import sharding


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist
    from oracle import recurrence

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert sharding.rank_env() == (rank, world, rank)
        # a rank's own time and units -> job-wide figures
        ms, units = sharding.aggregate(10.0 * (rank + 1), 1000 + rank)
        assert ms == 10.0 * world
        assert units == sum(1000 + r for r in range(world))
        assert sharding.throughput(units, ms) == units / (ms * 1e-3)

        # weak scaling: every rank draws its own batch
        cfg = gen.Config("tiny", 3, 128, 2, 16, 16, 64, "f32", True, False, seed=5)
        mine = gen.make_chunk_inputs(cfg, seed=sharding.rank_seed(cfg.seed, rank))
        digest = torch.tensor([float(np.abs(mine["q"]).sum())], dtype=torch.float64)
        both = [torch.zeros_like(digest) for _ in range(world)]
        dist.all_gather(both, digest)
        assert len({float(t.item()) for t in both}) == world, "ranks drew the same batch"

        # strong split of one global batch: each rank runs the oracle on its slice
        full = gen.make_chunk_inputs(cfg, seed=cfg.seed)
        lo, hi = sharding.batch_slice(cfg.B, rank, world)
        part = {n: (v[lo:hi] if isinstance(v, np.ndarray) and v.shape[:1] == (cfg.B,) else v) for n, v in full.items()}
        o, hT = recurrence.forward(part["q"], part["k"], part["v"], part["beta"], part["alpha"], part["lam"], part["h0"])
        np.save(os.path.join(out_dir, "o_%d.npy" % rank), o)
        np.save(os.path.join(out_dir, "hT_%d.npy" % rank), hT)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_batch_slices_cover_and_are_disjoint():
    for B in (1, 2, 7, 8, 64):
        for world in (1, 2, 3, 8):
            got = []
            for r in range(world):
                lo, hi = sharding.batch_slice(B, r, world)
                assert 0 <= lo <= hi <= B
                got += list(range(lo, hi))
            assert got == list(range(B))
            sizes = [sharding.batch_slice(B, r, world) for r in range(world)]
            assert max(h - l for l, h in sizes) - min(h - l for l, h in sizes) <= 1
    with pytest.raises(ValueError):
        sharding.batch_slice(4, 2, 2)


def test_aggregate_without_process_group_is_identity():
    assert sharding.aggregate(3.5, 77) == (3.5, 77)
    assert sharding.rank_seed(11, 0) == 11 and sharding.rank_seed(11, 3) == 14


@pytest.mark.timeout(300)
def test_two_gloo_ranks(tmp_path):
    from oracle import recurrence

    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    cfg = gen.Config("tiny", 3, 128, 2, 16, 16, 64, "f32", True, False, seed=5)
    full = gen.make_chunk_inputs(cfg, seed=cfg.seed)
    o, hT = recurrence.forward(full["q"], full["k"], full["v"], full["beta"], full["alpha"], full["lam"], full["h0"])
    o_parts = np.concatenate([np.load(tmp_path / ("o_%d.npy" % r)) for r in range(world)], axis=0)
    h_parts = np.concatenate([np.load(tmp_path / ("hT_%d.npy" % r)) for r in range(world)], axis=0)
    assert np.array_equal(o_parts, o)
    assert np.array_equal(h_parts, hT)

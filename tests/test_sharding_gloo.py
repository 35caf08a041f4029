"""Host-side multi-rank logic on CPU: world size 2 over gloo (no GPU, no data-path collective)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2411_05289_b200 import sharding


def test_shards_partition_the_batch():
    for batch in (0, 1, 2, 7, 64, 255, 1024):
        for world in (1, 2, 3, 8):
            sh = sharding.all_shards(batch, world)
            assert sh[0][0] == 0 and sh[-1][1] == batch
            for (a, b), (c, d) in zip(sh, sh[1:]):
                assert b == c and b >= a
            sizes = [b - a for a, b in sh]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.sequence_shard(4, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, batch, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import workloads

        cfg = workloads.Config("t", batch, 3, 64, "fp32", None, 2.0, 1.0, 1.0, seed=5)
        a, b = sharding.sequence_shard(batch, rank, world)
        # every rank builds only its own sequences; per-sequence seeding makes that possible
        lp, _ = workloads.host_logits(cfg, range(a, b)) if b > a else (np.zeros((0, 3, 64), np.float32), None)
        local = torch.from_numpy(lp.sum(axis=(1, 2)).astype(np.float64)).reshape(-1, 1)
        full = sharding.gather_per_sequence(local, batch)
        slow = sharding.max_over_ranks(1.0 + rank)
        q.put((rank, full.numpy().copy(), slow))
    finally:
        dist.destroy_process_group()


def test_two_ranks_gather_and_time():
    import workloads

    batch, world = 7, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, batch, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = workloads.Config("t", batch, 3, 64, "fp32", None, 2.0, 1.0, 1.0, seed=5)
    lp, _ = workloads.host_logits(cfg)
    want = lp.sum(axis=(1, 2)).astype(np.float64).reshape(-1, 1)
    for rank, full, slow in got:
        np.testing.assert_allclose(full, want, rtol=1e-12)
        assert slow == 2.0  # the slowest rank's time, on every rank

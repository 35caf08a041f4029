"""The exchanges of the vocabulary-sharded driver over gloo, world size 2, on CPU tensors:
gather order, element-wise maximum, and the slice bookkeeping every rank derives."""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    import torch.distributed as dist

    from paper_2411_05289_b200 import vocab_sharded as vs

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        widths = [501, 499]
        shard = vs.shard_of_group(widths[rank])
        # a phase output: [B][N][8] with a rank-specific pattern, including the int-in-float lane
        stats = torch.full((2, 3, 8), float(rank + 1))
        stats[..., 2] = torch.tensor([0x7fffffff if rank else 12345], dtype=torch.int32).view(torch.float32)
        g = vs.all_gather_ranks(stats)
        cand = torch.full((2, 3, 2), -2, dtype=torch.int32)
        cand[rank, :, 0] = 100 + rank          # each rank owns the draws of one sequence
        m = vs.all_max(cand)
        q.put((rank, shard, g.numpy().view(np.int32).copy(), m.numpy().copy()))
    finally:
        dist.destroy_process_group()


def test_exchanges_world_size_2():
    import torch.multiprocessing as mp

    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted([q.get(timeout=120) for _ in procs], key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, g0, m0), (r1, s1, g1, m1) = res
    assert (s0.rank, s0.nranks, s0.id_offset, s0.vocab_total) == (0, 2, 0, 1000)
    assert (s1.rank, s1.nranks, s1.id_offset, s1.vocab_total) == (1, 2, 501, 1000)
    np.testing.assert_array_equal(g0, g1)                      # every rank holds the same gathered block
    assert g0.shape == (2, 2, 3, 8)
    one, two = np.float32(1.0).view(np.int32), np.float32(2.0).view(np.int32)
    assert (g0[0, ..., 0] == one).all() and (g0[1, ..., 0] == two).all()   # rank order
    assert (g0[0, ..., 2] == 12345).all() and (g0[1, ..., 2] == 0x7fffffff).all()   # bit patterns survive
    np.testing.assert_array_equal(m0, m1)
    assert (m0[0, :, 0] == 100).all() and (m0[1, :, 0] == 101).all() and (m0[..., 1] == -2).all()


def _slice_worker(rank, world, port, q):
    import torch.distributed as dist

    from paper_2411_05289_b200 import vocab_sharded as vs

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank builds the same full rows (the benchmark's vocabulary-sharded leg does so from a
        # common seed) and keeps its own id range
        g = torch.Generator().manual_seed(5)
        full = torch.randn((2, 3, 1001), generator=g)
        shard, mine = vs.slice_of_rank(full, rank, world)
        assert mine.is_contiguous() and mine.shape == (2, 3, 501 if rank == 0 else 500)
        assert vs.shard_of_group(mine.shape[-1]) == shard          # the ranks agree on the bookkeeping
        # the slices, gathered in rank order, are the full rows again (pad to a common width to gather)
        pad = torch.zeros((2, 3, 501))
        pad[..., : mine.shape[-1]] = mine
        parts = vs.all_gather_ranks(pad)
        back = torch.cat([parts[0], parts[1][..., :500]], dim=-1)
        q.put((rank, bool(torch.equal(back, full))))
    finally:
        dist.destroy_process_group()


def test_vocabulary_slices_of_the_bench_leg_world_size_2():
    import torch.multiprocessing as mp

    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_slice_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted([q.get(timeout=120) for _ in procs])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, True), (1, True)]


def test_even_shards_cover_the_vocabulary():
    from paper_2411_05289_b200 import vocab_sharded as vs

    for V, n in ((1000, 3), (128256, 8), (7, 8), (32000, 1)):
        sh = vs.even_shards(V, n)
        assert sum(w for _, w in sh) == V
        off = 0
        for s, w in sh:
            assert s.id_offset == off and s.vocab_total == V and s.nranks == n
            off += w

"""Batch sharding over ranks: rows are independent and the tree walk needs only one sequence's
rows, so sequences are split over GPUs and nothing on the data path crosses ranks."""
from __future__ import annotations

from typing import List, Tuple


def sequence_shard(batch: int, rank: int, world: int) -> Tuple[int, int]:
    """[start, stop) of the sequences rank `rank` of `world` owns: contiguous, sizes differ by at
    most one, earlier ranks take the larger shards."""
    if world < 1 or not (0 <= rank < world) or batch < 0:
        raise ValueError("bad shard request: batch=%d rank=%d world=%d" % (batch, rank, world))
    base, extra = divmod(batch, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def all_shards(batch: int, world: int) -> List[Tuple[int, int]]:
    return [sequence_shard(batch, r, world) for r in range(world)]


def gather_per_sequence(local, batch: int, group=None):
    """All-gather a per-sequence tensor ([local_batch, ...], shards as in sequence_shard) into
    [batch, ...] on every rank.  Works on any backend (gloo on CPU, NCCL on GPUs)."""
    import torch
    import torch.distributed as dist

    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    s0, s1 = sequence_shard(batch, rank, world)
    if local.shape[0] != s1 - s0:
        raise ValueError("local shard has %d sequences, expected %d" % (local.shape[0], s1 - s0))
    width = max(b - a for a, b in all_shards(batch, world))
    pad = torch.zeros((width,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[: local.shape[0]] = local
    parts = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad, group=group)
    out = [parts[r][: b - a] for r, (a, b) in enumerate(all_shards(batch, world))]
    return torch.cat(out, dim=0)


def max_over_ranks(value: float, device=None, group=None) -> float:
    """The slowest rank's time: what a multi-GPU measurement reports."""
    import torch
    import torch.distributed as dist

    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())

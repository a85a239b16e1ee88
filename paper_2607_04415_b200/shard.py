"""Query sharding for multi-GPU runs: queries are independent, so rank r of `world` takes a
contiguous slice and owns a private page cache, request ring and proxy.  No data-path
collective exists; results are gathered only if the caller wants them in one place."""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_range(nq: int, rank: int, world: int):
    """Half-open [begin, end) of the queries rank `rank` searches (sizes differ by at most 1)."""
    base, rem = divmod(nq, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def gather_results(local: torch.Tensor, nq: int):
    """All-gather per-rank result rows (ragged along dim 0) into the global [nq, ...] order."""
    world, rank = dist.get_world_size(), dist.get_rank()
    sizes = [shard_range(nq, r, world)[1] - shard_range(nq, r, world)[0] for r in range(world)]
    pad = max(sizes)
    buf = torch.zeros((pad,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    buf[: local.shape[0]] = local
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf)
    return torch.cat([p[:s] for p, s in zip(parts, sizes)], 0)

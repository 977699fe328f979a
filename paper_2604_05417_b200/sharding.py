"""Batch sharding of the draft-verify round across ranks (one process per GPU).

The B sequences are independent bandit instances with per-sequence random-number counters, so the
path shards with no data-path collective: rank r owns a contiguous block of sequences and creates
its context with ``sequence_base`` = the global id of its first sequence, which makes the sharded
results identical to the unsharded ones.  Only reporting crosses ranks: the verified-token count is
summed and the step time is the maximum over ranks.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_range(batch: int, rank: int, world: int) -> Tuple[int, int]:
    """[first, last) global sequence ids of `rank` when `batch` sequences are split over `world` ranks:
    contiguous blocks whose sizes differ by at most one, the larger blocks first."""
    if world < 1 or not (0 <= rank < world) or batch < 0:
        raise ValueError("bad shard request: batch=%d rank=%d world=%d" % (batch, rank, world))
    base, extra = divmod(batch, world)
    first = rank * base + min(rank, extra)
    return first, first + base + (1 if rank < extra else 0)


def reduce_report(tokens: int, seconds: float, device=None) -> Tuple[int, float]:
    """Whole-job figures of a timed region: tokens summed over ranks, time = the slowest rank's."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return int(tokens), float(seconds)
    tok = torch.tensor([int(tokens)], dtype=torch.int64, device=device)
    sec = torch.tensor([float(seconds)], dtype=torch.float64, device=device)
    dist.all_reduce(tok, op=dist.ReduceOp.SUM)
    dist.all_reduce(sec, op=dist.ReduceOp.MAX)
    return int(tok.item()), float(sec.item())


def gather_outputs(local: torch.Tensor, batch: int) -> torch.Tensor:
    """Optional: every rank gets the [batch, ...] tensor assembled from the ranks' blocks (rank order)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return local
    world = dist.get_world_size()
    sizes = [hi - lo for lo, hi in (shard_range(batch, r, world) for r in range(world))]
    pad = max(sizes)                                   # all_gather wants equal shapes: pad the smaller blocks
    mine = torch.zeros((pad,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    mine[: local.shape[0]] = local
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine)
    return torch.cat([part[:n] for part, n in zip(parts, sizes)], dim=0)

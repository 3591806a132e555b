"""Host-side logic of the multi-GPU build: sequences are sharded across ranks (data parallel), each rank
accumulates its own statistics, one exchange sums them, the maps are solved in per-rank slices and gathered.

Only torch.distributed plumbing lives here (no arithmetic of the method beyond the sum the exchange performs).
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def shard_range(n: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous, balanced [begin, end) of n items for this rank (first n % world ranks get one more)."""
    base, rem = divmod(n, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def shard_chunks(n_chunks: int, rank: int, world: int) -> List[int]:
    """Chunk indices this rank streams when a fixed calibration set is split (strong scaling)."""
    a, b = shard_range(n_chunks, rank, world)
    return list(range(a, b))


def exchange_statistics(G: torch.Tensor, C: torch.Tensor, n_tokens: int, group=None) -> int:
    """Sum the per-rank statistics in place on every rank and return the global token count.
    Statistics are additive over any partition of the tokens, so this is the only data-path exchange."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return n_tokens
    dist.all_reduce(G, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(C, op=dist.ReduceOp.SUM, group=group)
    n = torch.tensor([n_tokens], dtype=torch.int64, device=G.device)
    dist.all_reduce(n, op=dist.ReduceOp.SUM, group=group)
    return int(n.item())


def gather_maps(Wb_local: torch.Tensor, n_maps: int, group=None) -> torch.Tensor:
    """Wb_local: [n_lambda][maps of this rank][p][d] for the rank's shard_range of maps -> full [n_lambda][n_maps][p][d]."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return Wb_local
    world = dist.get_world_size(group)
    nl, _, p, d = Wb_local.shape
    parts = []
    for r in range(world):
        a, b = shard_range(n_maps, r, world)
        parts.append(torch.empty(nl, b - a, p, d, dtype=Wb_local.dtype, device=Wb_local.device))
    dist.all_gather(parts, Wb_local.contiguous(), group=group) if len({x.shape for x in parts}) == 1 else \
        _all_gather_uneven(parts, Wb_local, group)
    return torch.cat(parts, dim=1)


def _all_gather_uneven(parts: List[torch.Tensor], mine: torch.Tensor, group) -> None:
    rank = dist.get_rank(group)
    for r, buf in enumerate(parts):
        if r == rank:
            buf.copy_(mine)
        dist.broadcast(buf, src=dist.get_global_rank(group, r) if group is not None else r, group=group)

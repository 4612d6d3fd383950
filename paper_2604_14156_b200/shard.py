"""Token sharding across ranks (one process per GPU).

The measure -> recover -> execute step treats every token independently, so a decode batch shards
over ranks with no collective on the data path: each rank holds all weights and runs the step on
its own slice of the tokens.  The only communication is control-plane: a barrier around timed
regions and a MAX reduction of the per-rank elapsed time.
"""
from __future__ import annotations

from typing import Tuple

import torch


def token_slice(n_tokens: int, world: int, rank: int) -> Tuple[int, int]:
    """[begin, end) of the tokens rank `rank` owns: contiguous, sizes differing by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_tokens, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def batch_stream(rank: int, j: int, per_rank: int) -> int:
    """Index of the j-th synthetic token batch of a rank (distinct batches on distinct ranks)."""
    return rank * per_rank + j


def max_over_ranks(value: float, device="cpu") -> float:
    """MAX over ranks of a scalar (elapsed time); identity without a process group."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_rows(local: torch.Tensor, n_tokens: int) -> torch.Tensor:
    """All ranks' token rows concatenated in rank order (for callers that want the full batch back)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return local
    world = dist.get_world_size()
    sizes = [token_slice(n_tokens, world, r) for r in range(world)]
    width = max(e - b for b, e in sizes)
    pad = torch.zeros((width,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[: local.shape[0]] = local
    out = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(out, pad)
    return torch.cat([o[: e - b] for o, (b, e) in zip(out, sizes)], dim=0)

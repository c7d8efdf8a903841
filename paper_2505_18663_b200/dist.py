"""Host-side plumbing of the multi-GPU (data-parallel) mode.

Tokens are independent in both stages of the path, so N GPUs simply take disjoint sets of
tokens with replicated packed weights: there is no data-path collective.  What remains is
bookkeeping: which tokens a rank owns, and the max-over-ranks of a timing.
"""
from __future__ import annotations

from typing import Tuple


def shard_tokens(M: int, rank: int, world: int, align: int = 128) -> Tuple[int, int]:
    """Contiguous token range [start, stop) of `rank` when M tokens are split over `world`
    ranks.  Boundaries are multiples of `align` (the GEMM's token tile) except the last stop."""
    if world < 1 or not (0 <= rank < world) or M < 0:
        raise ValueError("bad rank/world/M")
    tiles = (M + align - 1) // align
    per, extra = divmod(tiles, world)
    first = rank * per + min(rank, extra)
    count = per + (1 if rank < extra else 0)
    return min(M, first * align), min(M, (first + count) * align)


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Max of a per-rank scalar (an elapsed time) over all ranks; identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: float, elapsed_ms: float, world: int) -> float:
    """Whole-job rate when every rank processed `units_per_rank` in (max over ranks) elapsed_ms."""
    return world * units_per_rank / (elapsed_ms * 1e-3)

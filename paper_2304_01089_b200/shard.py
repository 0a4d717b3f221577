"""Token sharding of the hot path across ranks (one process per GPU).

Tokens are independent in both kernels, so the path shards over tokens with replicated tables and
weights and needs no collective on the data path. The only communication is a barrier around the
timed region and a max over the ranks' elapsed times.
"""
from __future__ import annotations

from typing import Sequence, Tuple


def token_range(total_tokens: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous share of `total_tokens` for `rank` (strong-scaling split; the first
    `total_tokens % world` ranks take one token more)."""
    if not (0 <= rank < world) or total_tokens < 0:
        raise ValueError("bad rank / world / token count")
    base, extra = divmod(total_tokens, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(values_ms: Sequence[float], dist=None, device=None):
    """Element-wise maximum of each rank's timings (what a multi-rank measurement must report)."""
    import torch
    t = torch.tensor(list(values_ms), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_throughput(units_per_rank: float, world: int, elapsed_ms_max: float) -> float:
    """Whole-job units per second when every rank processes `units_per_rank` in the slowest
    rank's time (weak scaling)."""
    return world * units_per_rank / (elapsed_ms_max * 1e-3)

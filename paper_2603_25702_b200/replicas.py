"""Multi-GPU use of the decode step: independent replicas.

Sequences never interact in S2D2 (every quantity of the block sampler is per sequence), so more
GPUs mean more replicas of the engine, each with the full weights and its own sequences; there is
no collective on the data path.  The only cross-rank traffic is what a benchmark needs to report
one number: the slowest rank's time and the total of committed tokens.
"""
from __future__ import annotations

from typing import Tuple


def rank_prompt_seed(base_seed: int, rank: int) -> int:
    """Every replica decodes its own prompts: one seed per rank."""
    return base_seed + rank


def aggregate_over_ranks(dev_ms: float, wall_s: float, committed: int, device: str = "cuda") -> Tuple[float, float, int]:
    """(max device time, max wall time, total committed tokens) over the ranks of the default
    torch.distributed group; identity when no group is initialised."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return dev_ms, wall_s, committed
    t = torch.tensor([dev_ms, wall_s], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([committed], device=device, dtype=torch.float64)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), int(n[0])

"""Host-side helpers for running one replica of the layer workload per GPU (batch sharding, no data-path collective).

Sequences are independent through the whole DARE layer step, so N GPUs run N replicas; the only communication is
the barrier around the timed region and the max-over-ranks of the measured time.
"""
from __future__ import annotations

import os


def rank_info():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when launched plainly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def rank_seed(base_seed: int, rank: int) -> int:
    """Every replica draws its own hidden states (and weights): distinct seeds per rank."""
    return base_seed + 1000 * rank


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """The slowest rank's figure, on every rank (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step: int, world: int, ms_per_step: float) -> float:
    """Units per second of the whole job: every rank processed `units_per_rank_per_step` in `ms_per_step`."""
    return world * units_per_rank_per_step / (ms_per_step * 1e-3)

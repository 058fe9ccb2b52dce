"""The little that several GPUs need: ranks decode disjoint batch shards and share nothing on
the data path, so the only collectives are the barrier and the MAX of the measured time."""
from __future__ import annotations

import os


def env_rank():
    """(rank, local_rank, world_size) as torchrun exports them; (0, 0, 1) when run alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def max_over_ranks(value: float, device="cpu") -> float:
    """MAX of a per-rank scalar over the default process group (identity without one)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: int, world_size: int, ms_max: float) -> float:
    """Units all ranks processed per second, given the slowest rank's time in ms."""
    return units_per_rank * world_size / (ms_max * 1e-3)

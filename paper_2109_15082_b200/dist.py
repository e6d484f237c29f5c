"""Host-side helpers for running one independent module replica per GPU ("replicas only": the
reconstruction step built here has no exchange between devices, so there is no collective on
the data path; torch.distributed is used for the barrier and for the max of the timings)."""
from __future__ import annotations

import os


def env_rank():
    """(rank, world_size, local_rank) from the torchrun environment; (0, 1, 0) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_seed(rank: int, base: int = 0) -> int:
    """Each replica draws its own weights and calibration set."""
    return base + rank


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's time (all ranks get it).  Works on any initialised backend."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def whole_job_rate(units_per_step_per_rank: int, steps: int, world: int, ms: float) -> float:
    """Aggregate units/s of `world` replicas that all ran `steps` steps within `ms` (the max over ranks)."""
    return world * units_per_step_per_rank * steps / (ms * 1e-3)

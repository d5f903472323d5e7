"""Multi-rank plumbing of the benchmark (replicas only: patch construction has no data-path collective).

Each rank builds the patch of its own context on its own GPU; the only communication is the barrier
around the timed region and the max-over-ranks of the measured time.  Kept free of CUDA so that it can be
exercised with the gloo backend on CPU."""
from __future__ import annotations

import os


def env_ranks():
    """(world_size, rank, local_rank) from the torchrun environment; (1, 0, 0) outside it."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_seed(base_seed: int, rank: int) -> int:
    """Every replica draws its own context: seed + rank."""
    return int(base_seed) + int(rank)


def max_over_ranks(value: float, device="cpu") -> float:
    """Max of a scalar over all ranks (identity when no process group is initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(ms_per_step_max: float, world: int) -> float:
    """ms per context of the whole job: `world` contexts are built in the time of the slowest rank."""
    return float(ms_per_step_max) / max(int(world), 1)

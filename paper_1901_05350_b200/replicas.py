"""Replica bookkeeping for multi-GPU runs.

The forward pass has no exchange step: images are independent and the weights are replicated, so N
GPUs run N independent replicas of the same batch (weak scaling) and nothing crosses NVLink on the
data path.  What ranks do share is timing: a barrier on both sides of the timed region and the
maximum of the per-rank device times.  These helpers hold that logic so that it can be exercised on
CPU with the gloo backend.
"""
from __future__ import annotations

import os


def env_rank_world():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) without it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of `value` over all ranks (the value itself when no process group is up)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def whole_job_throughput(units_per_rank_per_step: int, steps: int, elapsed_ms_this_rank: float, device=None) -> float:
    """Units per second of the whole job: every rank processed `units_per_rank_per_step * steps`
    units, and the job took as long as its slowest rank."""
    import torch.distributed as dist

    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    slowest_ms = max_over_ranks(elapsed_ms_this_rank, device)
    return world * units_per_rank_per_step * steps / (slowest_ms * 1e-3)

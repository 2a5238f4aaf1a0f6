"""One process per GPU: the little host logic the replicas share.

The path has no exchange step, so ranks never trade payload. What they do share: which batch a
rank works on (same shape, its own seed), a barrier around the timed region, the maximum of the
per-rank times, and the whole-job throughput computed from it."""
from __future__ import annotations

import os


def rank_env():
    """(rank, world_size, local_rank) from the launcher's environment (1 process = 1 GPU)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def workload_config_id(base_config: int, rank: int) -> int:
    """Seed stream of a rank's batch: every rank gets a batch of the same shape but its own
    draw (weak scaling: per-GPU work is fixed)."""
    return base_config + 100 * rank


def max_over_ranks(value: float, device=None) -> float:
    """Largest value over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(units_all_ranks: float, ms_max: float) -> float:
    """Units per second of the whole job: everything all ranks processed over the slowest rank's
    time."""
    return units_all_ranks / (ms_max * 1e-3)

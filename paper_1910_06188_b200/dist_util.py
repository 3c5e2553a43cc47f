"""Host-side plumbing for running the path on several GPUs of one node.

The quantised path needs no data-path collective: token rows are independent once the scales are fixed, so
every rank processes its own batch with replicated weights and scales (weak scaling).  What is left is
bookkeeping: which batch a rank draws, the device-time maximum over ranks, and the whole-job throughput.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(world_size, rank, local_rank) from the torchrun environment (1, 0, 0 when launched directly)."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_config(config: int, rank: int) -> int:
    """Seed family of a rank's batch: rank 0 uses the configuration's own seeds, rank r a disjoint family."""
    return int(config) + 100 * int(rank)


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar (elapsed device time) over all ranks; the value itself without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms_per_step: float) -> float:
    """Units per second of the whole job: every rank processes `units_per_rank` per step, the step takes the
    slowest rank's time."""
    return world * units_per_rank / (ms_per_step * 1e-3)

"""Data-parallel replicas: the layer shards by tokens with no exchange between ranks, so N GPUs run
N independent replicas (same parameters, a different batch each).  This module holds the little
host logic that exists: which batch a rank draws, and how per-rank timings become one whole-job
number (the slowest rank bounds the job)."""
from __future__ import annotations

import dataclasses
import os


def env_rank():
    """(rank, local_rank, world_size) as torchrun exports them; (0, 0, 1) when run directly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def rank_workload(wl, rank: int):
    """Workload whose batch streams (hidden states, upstream gradient) are rank-specific.  The
    parameter streams depend only on `wl.seed`, which callers keep for the weights."""
    return wl if rank == 0 else dataclasses.replace(wl, seed=wl.seed + 1000 * rank)


def max_over_ranks(value: float, device="cpu") -> float:
    """MAX all-reduce of one float over the default process group (identity without a group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def whole_job_rate(units_per_rank: int, world: int, ms_per_step_max: float) -> float:
    """Units per second of the whole job: every rank processes `units_per_rank` per step and the
    step takes as long as the slowest rank."""
    return world * units_per_rank / (ms_per_step_max * 1e-3)

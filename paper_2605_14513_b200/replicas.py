"""Multi-GPU plumbing of the benchmark: independent replicas, one process per GPU.

Every (batch, head) row of the hot path is independent and the library is a single-GPU kernel
library, so nothing is exchanged on the data path ("replicas only").  What the ranks do share is
the timing protocol: a barrier on both sides of the timed region, the maximum of the per-rank
device times, and the whole-job value derived from it.  These helpers hold exactly that and work on
any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank_world():
    """(rank, local_rank, world_size) from the torchrun environment (1 process = 1 GPU)."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` over all ranks (the job is as slow as its slowest replica)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def job_ms_per_layer_step(ms_per_step_slowest: float, world: int) -> float:
    """Whole-job time per layer-step: `world` replicas finish `world` layer-steps in the time the
    slowest replica needs for one (weak scaling: per-GPU work is fixed)."""
    return ms_per_step_slowest / float(world)

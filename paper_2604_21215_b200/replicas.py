"""Bookkeeping for running independent replicas of the workload on several GPUs.

The path shards over the batch only (sequences are independent), so N GPUs run N replicas with no
exchange on the data path.  What is shared is timing: a barrier around the timed region and the
maximum of the per-rank device times.  The same code runs under gloo on CPU (tests) and nccl on GPUs.
"""
from __future__ import annotations

from typing import Sequence


def world_info(env) -> tuple:
    """(world_size, rank, local_rank) from the launcher's environment."""
    return int(env.get("WORLD_SIZE", "1")), int(env.get("RANK", "0")), int(env.get("LOCAL_RANK", "0"))


def max_over_ranks(values: Sequence[float], device=None):
    """Element-wise maximum of `values` over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def aggregate_tokens_per_s(tokens_per_rank_step: int, steps: int, world: int, slowest_total_ms: float) -> float:
    """Whole-job throughput of `world` replicas: all ranks' tokens over the slowest rank's time."""
    return world * tokens_per_rank_step * steps / (slowest_total_ms * 1e-3)

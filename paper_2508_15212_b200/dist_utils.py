"""Multi-process plumbing of the benchmark: one process per GPU, no data-path collective.

The (sequence, KV head) units of the method are independent, so N GPUs run N disjoint sets of units
(weak scaling).  The only communication is the barrier around the timed region and the max-over-ranks of
the measured time.
"""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch


def env_ranks() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment; (0, 1, 0) when not launched."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init_process_group(backend: str, device: Optional[torch.device] = None):
    """Initialise torch.distributed from the environment (MASTER_ADDR/PORT, RANK, WORLD_SIZE).
    Returns the module, or None for a single process."""
    rank, world, _ = env_ranks()
    if world <= 1:
        return None
    import torch.distributed as dist
    kwargs = {}
    if backend == "nccl" and device is not None:
        kwargs["device_id"] = device
    dist.init_process_group(backend, rank=rank, world_size=world, **kwargs)
    return dist


def max_over_ranks(value: float, dist, device="cpu") -> float:
    """The slowest rank's time: what a multi-GPU step costs."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_seed_offset(rank: int, index: int = 0) -> int:
    """Distinct data per rank (and per copy / layer index within the rank)."""
    return rank * 64 + index


def aggregate_throughput(per_rank_units: float, world: int, seconds: float) -> float:
    """Whole-job rate: every rank processed `per_rank_units` in `seconds` (the max over ranks)."""
    return per_rank_units * world / seconds

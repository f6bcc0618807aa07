"""Multi-GPU plumbing: independent replicas of the per-GPU batch, no data-path collective.

Cache units never exchange data (every step of the path, eviction included, is local to a
unit), so N GPUs run N replicas of the batch, each on its own seeded trace.  The only
communication is for measurement: a barrier around the timed region and the maximum of
the per-rank device times.  Works with any torch.distributed backend (NCCL on GPUs, gloo
in the CPU tests).
"""
from __future__ import annotations

import os
from typing import Optional, Tuple


def rank_env() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) without one."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def replica_seed(seed: int, rank: int) -> int:
    """Seed of rank's trace: replicas see different data of the same distribution."""
    return int(seed) + 1000 * int(rank)


def init(backend: str, device=None):
    """Join the process group when launched with more than one rank; returns the module or None."""
    _, _, world = rank_env()
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        if device is not None:
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)
    return dist


def barrier(dist, sync=None) -> None:
    """Device synchronise (if given), then a barrier over all ranks, then synchronise again."""
    if sync is not None:
        sync()
    if dist is not None:
        dist.barrier()
        if sync is not None:
            sync()


def max_over_ranks(value: float, dist, device="cpu") -> float:
    """The largest of the ranks' values (the job is as slow as its slowest replica)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_second(batch_per_gpu: int, steps: int, world: int, ms_max: float) -> float:
    """Whole-job decode throughput: every replica advances its batch by `steps` tokens in ms_max."""
    return world * batch_per_gpu * steps / (ms_max * 1e-3)

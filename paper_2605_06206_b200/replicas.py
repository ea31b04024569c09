"""Rank plumbing of the benchmark's N > 1 mode.

The FoE block path does not shard: with N GPUs the benchmark runs N independent replicas (one process per GPU)
and there is no collective on the data path.  The only communication is around the timed region: a barrier on
both sides and the maximum of the per-rank times, from which the whole-job throughput follows.  The functions
work with any torch.distributed backend ("nccl" on GPUs, "gloo" on CPU for the tests).
"""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch
import torch.distributed as dist


def world() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment (1 process: 0, 1, 0)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device: Optional[torch.device] = None) -> bool:
    """Join the process group when WORLD_SIZE > 1.  Returns True if a group was created."""
    rank, size, _ = world()
    if size <= 1:
        return False
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    kw = {}
    if backend == "nccl" and device is not None:
        kw["device_id"] = device
    dist.init_process_group(backend, rank=rank, world_size=size, **kw)
    return True


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar (the slowest replica decides the job's time)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank_step: int, steps: int, ms_total_local: float, device="cpu") -> Tuple[float, float]:
    """(units per second over all replicas, ms per step) from this rank's time for `steps` steps: the time is the
    maximum over ranks, the units are those of all ranks together (weak scaling: per-rank work is fixed)."""
    _, size, _ = world()
    ms = max_over_ranks(ms_total_local, device)
    return size * units_per_rank_step * steps / (ms * 1e-3), ms / steps


def shutdown() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()

"""Host logic of the multi-GPU benchmark mode: independent replicas, one process per GPU.

The forward path has no exchange step, so N GPUs run N replicas of the workload; the only
communication is bookkeeping: a barrier around the timed region, the slowest rank's time and the
total number of units processed.  Works with any torch.distributed backend (NCCL on GPUs, gloo on
CPU in the tests).
"""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch
import torch.distributed as dist


def env_rank() -> Tuple[int, int, int]:
    """(rank, local rank, world size) from the launcher's environment (1 process = rank 0 of 1)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device: Optional[torch.device] = None) -> bool:
    """Joins the process group when launched with more than one rank.  Returns True if it did."""
    _, _, world = env_rank()
    if world <= 1:
        return False
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if backend == "nccl" and device is not None:
        dist.init_process_group(backend, device_id=device)
    else:
        dist.init_process_group(backend)
    return True


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate(local_ms: float, local_units: int, device: torch.device) -> Tuple[float, int]:
    """(time of the slowest rank, units processed by all ranks)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(local_ms), int(local_units)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([int(local_units)], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), int(u.item())


def throughput(local_ms_per_step: float, local_units_per_step: int, device: torch.device) -> Tuple[float, float]:
    """Whole-job units per second and the slowest rank's ms per step."""
    ms, units = aggregate(local_ms_per_step, local_units_per_step, device)
    return units / (ms * 1e-3), ms


def finish() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()

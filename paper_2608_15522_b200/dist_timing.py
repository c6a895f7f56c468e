"""Multi-process plumbing of the benchmark: rank set-up, barrier, and max-over-ranks of timings.

The path itself has no collective (every GPU runs an independent replica of the layer); these helpers only
bracket the timed region and combine the per-rank times.  They work with NCCL on GPUs and with gloo on CPU
(the latter is what the CPU test suite exercises).
"""
from __future__ import annotations

import os
from typing import Optional, Sequence

import torch


def world() -> tuple:
    """(rank, local_rank, world_size) from the launcher's environment (torchrun), defaults for a plain run."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device: Optional[torch.device] = None):
    """Initialises torch.distributed when WORLD_SIZE > 1; returns the module or None."""
    _, _, size = world()
    if size <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        kwargs = {}
        if backend == "nccl" and device is not None:
            kwargs["device_id"] = device
        dist.init_process_group(backend, **kwargs)
    return dist


def barrier(dist, device: Optional[torch.device] = None) -> None:
    if device is not None and device.type == "cuda":
        torch.cuda.synchronize(device)
    if dist is not None:
        dist.barrier()
    if device is not None and device.type == "cuda":
        torch.cuda.synchronize(device)


def max_over_ranks(dist, values: Sequence[float], device: Optional[torch.device] = None) -> list:
    """Element-wise maximum of a short list of per-rank numbers (times in ms)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device if device is not None else "cpu")
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_rate(units_per_rank: float, world_size: int, max_ms: float) -> float:
    """Units all ranks processed divided by the slowest rank's time (weak scaling: same units on every rank)."""
    return units_per_rank * world_size / (max_ms * 1e-3)

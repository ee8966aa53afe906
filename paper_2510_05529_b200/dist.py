"""Multi-process plumbing of the benchmark: the hot path itself never communicates.

Every (layer, sequence, KV head) of the cache is independent, so N GPUs run N independent sequences
(replicas). torch.distributed is used only to line the ranks up (barrier) and to take the maximum of
their timings; `nccl` on GPUs, `gloo` in the CPU tests.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def world():
    """(rank, world_size, local_rank) from the launcher's environment (1 process if unset)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device: torch.device | None = None) -> bool:
    """Join the process group if there is more than one rank. Returns True when a group exists."""
    _, n, _ = world()
    if n <= 1:
        return False
    if not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, **kw)
    return True


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(values, device: torch.device | str = "cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity for a single process)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_rate(units_per_rank: float, n_ranks: int, seconds_max_over_ranks: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return units_per_rank * n_ranks / seconds_max_over_ranks


def finish():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()

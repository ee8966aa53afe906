"""Multi-process plumbing of the benchmark: the hot path itself never communicates.

Every (layer, sequence, KV head) of the cache is independent (the method is stated per attention
head, Section IV-A), so N GPUs either run N independent sequence sets (replicas) or split the KV
heads of the same sequences between them (`shard_heads`): in both layouts no rank ever needs
another rank's data. torch.distributed is used only to line the ranks up (barrier) and to take the
maximum of their timings; `nccl` on GPUs, `gloo` in the CPU tests.
"""
from __future__ import annotations

import os
from typing import NamedTuple

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


class HeadShard(NamedTuple):
    """The heads one rank owns: KV heads [kv_begin, kv_begin + n_kv) and their query heads
    [q_begin, q_begin + n_q) of the unsharded model."""
    kv_begin: int
    n_kv: int
    q_begin: int
    n_q: int


def shard_heads(n_q_heads: int, n_kv_heads: int, rank: int, world: int, head_dim: int = 128) -> HeadShard:
    """Which heads rank `rank` of `world` owns when the ranks split the heads of the same sequences.

    Contiguous blocks of KV heads, each with all the query heads of its group (query head h reads KV
    head h // (Hq / Hkv), so a group is never cut), the same number on every rank. 64-wide heads
    travel in pairs through the 128-channel kernels, so a rank then takes an even number of KV heads.
    Raises ValueError when the heads do not divide that way. The ranks' slices are disjoint and their
    union is the whole head set; in the [.., Hq, d] output of the unsharded model rank r's rows are
    [q_begin, q_begin + n_q), so concatenating the ranks' outputs along the head axis in rank order
    gives the unsharded tensor."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("rank %d outside [0, %d)" % (rank, world))
    if n_kv_heads < 1 or n_q_heads % n_kv_heads:
        raise ValueError("%d query heads do not group over %d KV heads" % (n_q_heads, n_kv_heads))
    if n_kv_heads % world:
        raise ValueError("%d KV heads do not divide over %d ranks" % (n_kv_heads, world))
    n_kv = n_kv_heads // world
    if head_dim == 64 and n_kv % 2:
        raise ValueError("64-wide heads are cached in pairs: %d KV heads per rank is odd" % n_kv)
    gq = n_q_heads // n_kv_heads
    return HeadShard(rank * n_kv, n_kv, rank * n_kv * gq, n_kv * gq)


def take_heads(t: torch.Tensor, begin: int, n: int, axis: int = -2) -> torch.Tensor:
    """This rank's heads of a tensor whose `axis` is the head axis (K, V: [.., Hkv, d]; q, out: [.., Hq, d]),
    as a contiguous tensor. Data movement only."""
    return t.narrow(axis, begin, n).contiguous()


def finish():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()

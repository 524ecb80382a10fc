"""Host-side logic for running one workload's replicas on several GPUs.

Replicas never exchange state and all randomness is keyed by the global replica index, so a
network can be cut along the replica axis with no data-path collective: every process builds
a network for its slice with `replica_offset` set to the slice's first global index, and only
the counters are summed at the end (one small all-reduce).
"""
from __future__ import annotations

import numpy as np


def replica_shard(n_replicas: int, world_size: int, rank: int):
    """Contiguous slice [offset, offset + count) of `n_replicas` owned by `rank`; the first
    `n_replicas % world_size` ranks get one extra replica."""
    if not (0 <= rank < world_size):
        raise ValueError("rank out of range")
    base, extra = divmod(n_replicas, world_size)
    count = base + (1 if rank < extra else 0)
    offset = rank * base + min(rank, extra)
    return offset, count


def sum_counters(local_totals: np.ndarray, group=None) -> np.ndarray:
    """All-reduce (sum) of one counter record over the process group; identity without one."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return local_totals
    t = torch.from_numpy(np.ascontiguousarray(local_totals).view(np.int64).copy())
    if dist.get_backend(group) == "nccl":
        t = t.cuda()
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t.cpu().numpy().view(np.uint64)


def max_over_ranks(value: float, group=None) -> float:
    """Max of a per-rank elapsed time (timing rule for multi-GPU numbers)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64)
    if dist.get_backend(group) == "nccl":
        t = t.cuda()
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())

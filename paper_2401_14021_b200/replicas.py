"""Aggregation of independent replicas (one process per GPU).

The retrieval path does not shard: every rank owns a full copy of the corpus and answers its
own requests, and the only exchange between ranks is the bookkeeping below (a barrier around
the timed region, the slowest rank's time, the total number of queries). It works on any
torch.distributed backend; nothing here touches the data path.
"""
from typing import Sequence, Tuple

import torch


def world() -> Tuple[int, int]:
    """(rank, world size) of the initialised process group, (0, 1) without one."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def barrier() -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate(times_ms: Sequence[float], queries: int, device="cpu") -> Tuple[list, int]:
    """Whole-job figures from per-rank ones: element-wise MAX of the times (the job is done when
    its slowest replica is), SUM of the queries answered. Every rank gets the same result."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return [float(t) for t in times_ms], int(queries)
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    n = torch.tensor([int(queries)], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return t.tolist(), int(n.item())


def throughput(times_ms: Sequence[float], queries: int, device="cpu") -> list:
    """Queries per second of the whole job for each timed region."""
    t, n = aggregate(times_ms, queries, device)
    return [n / (ms * 1e-3) if ms > 0 else float("inf") for ms in t]

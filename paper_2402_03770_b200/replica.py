"""Multi-GPU plumbing: the compression path runs on one GPU, so several GPUs are independent
replicas (every rank compresses its own clients and aggregates them); ranks only meet at a
barrier and to agree on the slowest rank's time.  No data-path collective."""
from __future__ import annotations

from typing import List

import torch
import torch.distributed as dist


def replica_clients(rank: int, clients_per_rank: int) -> List[int]:
    """global client ids owned by `rank` (disjoint across ranks, so every replica has its own data)"""
    return list(range(rank * clients_per_rank, (rank + 1) * clients_per_rank))


def max_over_ranks(value: float, device: torch.device) -> float:
    """the largest `value` of any rank (the job's time is the slowest replica's)"""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: int, world_size: int, slowest_ms: float) -> float:
    """units all ranks processed per second"""
    return units_per_rank * world_size / (slowest_ms * 1e-3)

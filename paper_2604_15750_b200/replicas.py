"""Multi-GPU running of the block-step: replicas only.

Sequences are independent and the weights are read-only, so N GPUs run N independent replicas
over disjoint sequences (one process per GPU); the data path has no exchange step and no
collective.  What the ranks do share is bookkeeping for a measurement: a barrier around the
timed region, the slowest rank's time, and the sum of the committed tokens.  That bookkeeping
lives here so that it can be exercised on CPU (gloo) as well as on GPUs (nccl).
"""
from __future__ import annotations

import torch


def replica_seed(base_seed: int, rank: int) -> int:
    """Seed of the sequences replica `rank` draws (rank 0 keeps the workload's own seed)."""
    return base_seed + 1000 * rank


def combine(dist, times_ms, counts, device="cpu"):
    """Max over ranks of each time, sum over ranks of each count.  `dist` is torch.distributed
    (initialised) or None for a single process."""
    if dist is None:
        return [float(t) for t in times_ms], [int(c) for c in counts]
    t = torch.tensor([float(x) for x in times_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor([int(x) for x in counts], dtype=torch.int64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], [int(x) for x in c.tolist()]


def aggregate_throughput(total_count: int, slowest_ms: float) -> float:
    """Whole-job units per second: everything all ranks processed over the slowest rank's time."""
    return total_count / (slowest_ms * 1e-3)

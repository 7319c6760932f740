"""Multi-process plumbing of the benchmark: replicas only, no data-path collective.

The path does not shard (every rank steps its own replica), so the only exchange is the timing:
the slowest rank defines the step time, and the job's throughput is the sum of the units all ranks
processed divided by that time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def sum_over_ranks(values, device="cpu"):
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return [float(v) for v in t]


def aggregate_throughput(units_this_rank: float, ms_this_rank: float, device="cpu"):
    """(whole-job units per second, ms of the slowest rank)."""
    (ms,) = max_over_ranks([ms_this_rank], device)
    (units,) = sum_over_ranks([units_this_rank], device)
    return units / (ms * 1e-3), ms


def sync_layer_stats(stats, device="cpu"):
    """Cross-rank aggregate of the per-layer gradient sums (the paper's "distributed engine" step).

    stats: [L, 4] float64 rows {sum g, sum |g|, sum g^2, count} of this rank's local gradients, as
    returned by ``stq_layer_stats``.  All four columns are sums over elements, so the job-wide
    statistics are their sums over ranks; every rank then takes the same O(L) decision.  One
    all-reduce of 4L doubles on decision steps only; identity without a process group."""
    import numpy as np
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return np.asarray(stats, dtype=np.float64)
    t = torch.as_tensor(np.ascontiguousarray(stats, dtype=np.float64), device=device).clone()
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t.cpu().numpy()

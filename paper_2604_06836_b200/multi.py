"""Multi-process plumbing: replicas for the benchmark, and the host side of a sharded optimizer.

The benchmark runs replicas (every rank steps its own copy), so its only exchange is the timing:
the slowest rank defines the step time, and the job's throughput is the sum of the units all ranks
processed divided by that time.

A sharded optimizer (each rank keeps the quantized state of a slice of the parameters) needs no
data-path collective either, because quantization blocks are independent: ``partition`` cuts the
parameter list into per-rank element ranges on block boundaries, each rank steps its ranges as rows
of its own table, and on decision steps the per-layer sums are added over ranks
(``sync_layer_stats``, Sec. 3.1's distributed engine) so that every rank takes the same decision.
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


def partition(numels, world: int, align: int = 4096):
    """Cuts the concatenated parameter list into ``world`` contiguous shares of about equal size.

    Returns one list per rank of (tensor index, first element, end element).  A cut inside a tensor
    falls on a multiple of ``align`` elements from the tensor's start (the default, one kernel tile,
    is a multiple of every block size, so no quantization block is split and every range starts on a
    16-byte boundary of the packed codes for every width).  Ranges of one tensor on different ranks
    are disjoint and cover it; a rank may get no range when there is less work than ranks."""
    numels = [int(n) for n in numels]
    total = sum(numels)
    shares = [[] for _ in range(world)]
    # units: whole align-sized pieces (the ragged tail of a tensor belongs to its last piece)
    pieces = [max(1, (n + align - 1) // align) if n > 0 else 0 for n in numels]
    npieces = sum(pieces)
    done = 0            # pieces handed out so far
    rank = 0
    for l, (n, p) in enumerate(zip(numels, pieces)):
        first = 0       # piece index inside the tensor
        while first < p:
            # the rank's share ends at piece index round((rank+1) * npieces / world) of the whole list
            end_global = ((rank + 1) * npieces + world - 1) // world
            take = min(p - first, end_global - done)
            if take <= 0:
                rank += 1
                continue
            lo, hi = first * align, min(n, (first + take) * align)
            shares[rank].append((l, lo, hi))
            first += take
            done += take
    assert done == npieces and sum(hi - lo for sh in shares for _, lo, hi in sh) == total
    return shares

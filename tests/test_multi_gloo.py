"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, replicas only."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2604_06836_b200 import multi
    # rank 0 took 4 ms for 1000 units, rank 1 took 5 ms for 1000 units
    value, ms = multi.aggregate_throughput(1000.0, 4.0 + rank)
    mx = multi.max_over_ranks([float(rank), 10.0 - rank])
    dist.barrier()
    if rank == 0:
        torch.save({"value": value, "ms": ms, "mx": mx}, out)
    dist.destroy_process_group()


def test_two_rank_aggregation(tmp_path):
    out = str(tmp_path / "r0.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r = torch.load(out)
    assert r["ms"] == 5.0                              # the slowest rank defines the time
    assert abs(r["value"] - 2000.0 / 5e-3) < 1e-6      # all ranks' units over that time
    assert r["mx"] == [1.0, 10.0]


def test_single_process_is_identity():
    from paper_2604_06836_b200 import multi
    assert multi.aggregate_throughput(10.0, 2.0) == (5000.0, 2.0)

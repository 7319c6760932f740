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
    # per-layer statistics of two ranks holding different local gradients of the same 3 layers
    import numpy as np
    import oracle
    rng = np.random.default_rng(100 + rank)
    grads = [rng.normal(0, 1e-3 * (l + 1), 1000 + 10 * l).astype(np.float32) for l in range(3)]
    local = np.stack([oracle.grad_stats(g) for g in grads])
    synced = multi.sync_layer_stats(local)
    pol = oracle.new_policy(0.1, 100.0)
    bits, _ = oracle.decide(pol, synced, 10)
    dist.barrier()
    torch.save({"value": value, "ms": ms, "mx": mx, "synced": synced, "local": local, "bits": bits}, out + str(rank))
    dist.destroy_process_group()


def test_two_rank_aggregation(tmp_path):
    out = str(tmp_path / "r0.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r = torch.load(out + "0", weights_only=False)
    r1 = torch.load(out + "1", weights_only=False)
    assert r["ms"] == 5.0                              # the slowest rank defines the time
    assert abs(r["value"] - 2000.0 / 5e-3) < 1e-6      # all ranks' units over that time
    assert r["mx"] == [1.0, 10.0]
    # statistics: the sums add over ranks, every rank ends with the same numbers and the same decision
    import numpy as np
    np.testing.assert_allclose(r["synced"], r["local"] + r1["local"], rtol=1e-15)
    assert (r["synced"] == r1["synced"]).all() and (r["bits"] == r1["bits"]).all()
    assert (r["synced"][:, 3] == 2 * r["local"][:, 3]).all()


def test_single_process_is_identity():
    from paper_2604_06836_b200 import multi
    assert multi.aggregate_throughput(10.0, 2.0) == (5000.0, 2.0)

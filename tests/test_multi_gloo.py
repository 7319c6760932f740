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


# ---- sharded optimizer: each rank owns element ranges of the parameter list ------------------------------
def _shard_problem():
    """A small mixed-width problem; every process draws the same tensors from the same seeds."""
    import numpy as np
    from paper_2604_06836_b200 import workloads as W
    w = W.scaled(W.config("cfg2"), W.small_gpt2(d=72, n_layer=1, vocab=301, ctx=16), steps=3)
    bm, bv, _ = W.draw_bits(w)
    theta = [W.draw_param(w, i).numpy().copy() for i in range(len(w.shapes))]
    grads = [[W.draw_grad(w, i, t).numpy().copy() for i in range(len(w.shapes))] for t in (1, 2, 3)]
    return w, bm, bv, theta, grads


def _shard_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import numpy as np
    import oracle
    from paper_2604_06836_b200 import multi
    w, bm, bv, theta, grads = _shard_problem()
    mine = multi.partition(w.numels, world, align=256)[rank]
    th = [theta[l][lo:hi].copy() for l, lo, hi in mine]
    st = [oracle.new_state(hi - lo, w.block, int(bm[l]), int(bv[l])) for l, lo, hi in mine]
    pol = oracle.new_policy(0.1, 100.0)
    bits = None
    for t in (1, 2, 3):
        local = np.zeros((len(w.shapes), 4))
        for k, (l, lo, hi) in enumerate(mine):
            g = grads[t - 1][l][lo:hi]
            st[k], s = oracle.step(th[k], g, st[k], w.block, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                                   weight_decay=w.weight_decay, t=t, want_stats=True)
            local[l] += s
        synced = multi.sync_layer_stats(local)          # every step is a decision step while t < 5
        bits, _ = oracle.decide(pol, synced, t)
    dist.barrier()
    torch.save({"mine": mine, "theta": th, "states": st, "synced": synced, "bits": bits}, out + str(rank))
    dist.destroy_process_group()


def test_sharded_ranks_reproduce_the_single_process_step(tmp_path):
    """Two ranks step disjoint block ranges and add their per-layer sums: states and parameters equal
    the single-process result bit for bit, the statistics agree to rounding and both ranks take the
    single-process decision."""
    import numpy as np
    import oracle
    out = str(tmp_path / "s")
    mp.spawn(_shard_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    w, bm, bv, theta, grads = _shard_problem()
    L = len(w.shapes)
    st = [oracle.new_state(n, w.block, int(bm[l]), int(bv[l])) for l, n in enumerate(w.numels)]
    pol = oracle.new_policy(0.1, 100.0)
    for t in (1, 2, 3):
        stats = np.zeros((L, 4))
        for l in range(L):
            st[l], stats[l] = oracle.step(theta[l], grads[t - 1][l], st[l], w.block, lr=w.lr, beta1=w.beta1,
                                          beta2=w.beta2, eps=w.eps, weight_decay=w.weight_decay, t=t,
                                          want_stats=True)
        bits, _ = oracle.decide(pol, stats, t)
    seen = [0] * L
    ranks = [torch.load(out + str(r), weights_only=False) for r in range(2)]
    assert any(lo > 0 for r in ranks for _, lo, _ in r["mine"])        # some tensor is really split
    for r in ranks:
        np.testing.assert_allclose(r["synced"], stats, rtol=1e-12, atol=1e-300)
        assert (r["synced"][:, 3] == stats[:, 3]).all()
        assert (np.asarray(r["bits"]) == np.asarray(bits)).all()
        for k, (l, lo, hi) in enumerate(r["mine"]):
            seen[l] += hi - lo
            s, full = r["states"][k], st[l]
            assert (r["theta"][k] == theta[l][lo:hi]).all()
            for codes, whole, b in ((s.m_codes, full.m_codes, int(bm[l])), (s.v_codes, full.v_codes, int(bv[l]))):
                nbytes = ((hi - lo) * b + 7) // 8
                assert (codes[:nbytes] == whole[lo * b // 8: lo * b // 8 + nbytes]).all()
            nb = (hi - lo + w.block - 1) // w.block
            assert (s.m_scales[:nb].view(np.uint32) == full.m_scales[lo // w.block: lo // w.block + nb].view(np.uint32)).all()
            assert (s.v_scales[:nb].view(np.uint32) == full.v_scales[lo // w.block: lo // w.block + nb].view(np.uint32)).all()
    assert seen == list(w.numels)


def test_partition_covers_everything_on_block_boundaries():
    from paper_2604_06836_b200 import multi, workloads as W
    for numels, world in (([10, 5000, 3], 4), ([10], 4), (W.config("cfg2").numels, 8), (W.config("cfg5").numels, 8),
                          ([4096 * 7 + 1], 3), ([], 2)):
        shares = multi.partition(numels, world)
        assert len(shares) == world
        flat = sorted(r for sh in shares for r in sh)
        cover = [0] * len(numels)
        for l, lo, hi in flat:
            assert lo == cover[l] and lo % 4096 == 0 and lo < hi <= numels[l]
            cover[l] = hi
        assert cover == [int(n) for n in numels]
        # contiguous: a rank's ranges follow the previous rank's in list order
        order = [r for sh in shares for r in sh]
        assert order == flat
    sizes = [sum(hi - lo for _, lo, hi in sh) for sh in multi.partition(W.config("cfg5").numels, 8)]
    assert max(sizes) / min(sizes) < 1.01

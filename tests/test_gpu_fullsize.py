"""The benchmark configurations at full size, in the launch configuration bench.py times.

The oracle cannot step 1.5e9 parameters in seconds, so it follows a sample of quantization blocks of
every tensor (first, last, ragged tail, blocks next to tile boundaries, random ones): blocks are
independent given their inputs, so the sampled blocks are checked exactly as the small cases are
(codes and scales bit for bit, parameters to 1e-6 per step).  Statistics of tensors small enough are
checked against the oracle, the large ones against a float64 library reduction.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2604_06836_b200 import workloads as W   # noqa: E402
from paper_2604_06836_b200.runner import Job        # noqa: E402


def _need(gb):
    free, _ = torch.cuda.mem_get_info()
    if free < gb * 2 ** 30:
        pytest.skip(f"needs {gb} GiB of free device memory")


@pytest.mark.parametrize("name,gib,steps", [("cfg2", 4, 6), ("cfg3", 3, 6), ("cfg4", 14, 3), ("cfg5", 26, 3)])
def test_full_size_sampled_blocks(name, gib, steps):
    import harness as H
    import oracle
    _need(gib)
    w = W.config(name)
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv)
    so = H.SampledOracle(job, per_tensor=4, seed=1)
    so.compare(0.0, f"{name} init")
    for t in range(1, steps + 1):
        job.draw_grads(t)
        stats = (t == steps)
        so.step(t)
        job.step(t, stats=stats)
        so.compare(1e-6 * t, f"{name} t={t}")
    got = job.layer_stats()
    for i, g in enumerate(job.grads):
        if g.numel() <= (1 << 21):
            want = oracle.grad_stats(H.to_np(g))
        else:
            g64 = g.double()
            want = np.array([g64.sum().item(), g64.abs().sum().item(), (g64 * g64).sum().item(), g.numel()])
        H.assert_stats_close(got[i:i + 1], want[None, :], f"{name} stats tensor {i}")
    # memory accounting of the problem statement: sum over layers of 2 * N_l * b_l bits (+ scales)
    bits = sum(n * (int(a) + int(b)) for n, a, b in zip(w.numels, bm, bv))
    code_bytes = sum(s.m_codes.numel() + s.v_codes.numel() for s in job.states)
    assert bits / 8 <= code_bytes <= bits / 8 + 32 * job.L
    assert job.state_bytes() < 0.25 * 8 * w.total_params     # far below the fp32 states


def test_errors_are_reported_before_anything_runs():
    from paper_2604_06836_b200 import stq
    h = stq.Handle()
    n = 5000
    dev = "cuda"
    p = torch.zeros(n, device=dev)
    g = torch.zeros(n, device=dev)
    st = stq.alloc_state(n, 128, 8, 4, dev)
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, t=1)

    def code_of(row, **kw):
        try:
            h.step(stq.table([row]), **{**hp, **kw})
        except stq.StqError as e:
            return e.code
        return 0

    good = stq.make_row(n, 128, st, st, p, g, 0.01)
    assert code_of(good) == 0
    bad = stq.make_row(n, 100, st, st, p, g, 0.01)
    assert code_of(bad) == -3                                   # block
    bad = stq.make_row(n, 128, st, st, p, g, 0.01); bad.bits_m = 5
    assert code_of(bad) == -2                                   # width
    bad = stq.make_row(n, 128, st, st, p, g, 0.01); bad.param = None
    assert code_of(bad) == -1                                   # null
    bad = stq.make_row(n, 128, st, st, p, g, 0.01); bad.grad = g.data_ptr() + 4
    assert code_of(bad) == -4                                   # alignment
    bad = stq.make_row(n, 128, st, st, p, g, 0.01); bad.bits_m_out = 4
    assert code_of(bad) == -5                                   # in-place with a width change
    bad = stq.make_row(0, 128, st, st, p, g, 0.01)
    assert code_of(bad) == -6                                   # numel
    assert code_of(good, t=0) == -9                             # step index
    with pytest.raises(stq.StqError) as ei:
        h.layer_stats(1)
    assert ei.value.code == -10                                 # no statistics pending
    torch.cuda.synchronize()
    assert (p == 0).all()     # zero gradients, zero parameters: the one good step left them at zero
    h.device_status()


def test_checkpoint_resume_is_bit_identical():
    """State = caller-owned buffers + (t, widths): copying them is a checkpoint."""
    w = W.scaled(W.config("cfg2"), W.small_gpt2(), steps=6)
    bm, bv, _ = W.draw_bits(w)
    a = Job(w, bm, bv)
    for t in (1, 2, 3):
        a.draw_grads(t)
        a.step(t)
    b = Job(w, bm, bv)
    b.param_flat.copy_(a.param_flat)
    for sa, sb in zip(a.states, b.states):
        sb.m_codes.copy_(sa.m_codes); sb.m_scales.copy_(sa.m_scales)
        sb.v_codes.copy_(sa.v_codes); sb.v_scales.copy_(sa.v_scales)
    for t in (4, 5, 6):
        a.draw_grads(t); b.draw_grads(t)
        a.step(t); b.step(t)
    torch.cuda.synchronize()
    assert torch.equal(a.param_flat, b.param_flat)
    for sa, sb in zip(a.states, b.states):
        assert torch.equal(sa.m_codes, sb.m_codes) and torch.equal(sa.v_codes, sb.v_codes)
        assert torch.equal(sa.m_scales, sb.m_scales) and torch.equal(sa.v_scales, sb.v_scales)


def test_host_buffer_step_matches_device_step():
    """stq_step_host (host pointers, copies inside the call) against stq_step on device buffers."""
    from paper_2604_06836_b200 import stq
    w = W.scaled(W.config("cfg4"), W.small_gpt2(d=136, n_layer=2), steps=2)
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv)
    job.draw_grads(1)
    job.step(1)
    job.draw_grads(2)
    torch.cuda.synchronize()
    hp_ = job.param_flat.cpu().pin_memory()
    hg = job.grad_flat.cpu().pin_memory()
    rows, hstates = [], []
    for i, n in enumerate(job.numels):
        s = job.states[i]
        hs = stq.QState(s.m_codes.cpu().pin_memory(), s.m_scales.cpu().pin_memory(), s.bits_m,
                        s.v_codes.cpu().pin_memory(), s.v_scales.cpu().pin_memory(), s.bits_v)
        hstates.append(hs)
        o = job.offsets[i]
        rows.append(stq.make_row(n, job.block, hs, hs, hp_[o:o + n], hg[o:o + n], job.wd[i]))
    h2d, d2h = job.handle.step_host(stq.table(rows), **job.hp(2))
    job._tbl = None
    job.step(2)
    torch.cuda.synchronize()
    assert h2d > 0 and d2h > 0
    assert torch.equal(hp_, job.param_flat.cpu())
    for hs, s in zip(hstates, job.states):
        assert torch.equal(hs.m_codes, s.m_codes.cpu()) and torch.equal(hs.v_codes, s.v_codes.cpu())
        assert torch.equal(hs.m_scales, s.m_scales.cpu()) and torch.equal(hs.v_scales, s.v_scales.cpu())

"""The benchmark configurations at full size, in the launch configuration bench.py times.

Two kinds of comparison.  Every element: the oracle, spread over the host cores range by range, steps the
whole parameter list and every code byte, scale and parameter is compared (all steps of the two small
configurations; the first three steps of the two large ones, all three decision steps with statistics).
Sampled blocks: for the remaining steps of the large configurations, the fp16 workloads and the second
variant of the v quantizer the oracle follows a sample of quantization blocks of every tensor (first, last,
ragged tail, blocks next to tile boundaries, random ones); blocks are independent given their inputs, so
they are checked exactly as the small cases are.  Statistics of tensors small enough are checked against the
oracle, the large ones against a float64 library reduction.
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


@pytest.mark.parametrize("name,gib", [("cfg2", 4), ("cfg3", 3), ("cfg4", 14), ("cfg5", 26),
                                      ("gpt2_medium", 8), ("roberta_large", 8), ("vit_b32", 3),
                                      ("cfg3:pl", 3), ("cfg5:pl", 26)])
def test_full_size_sampled_blocks(name, gib):
    """Each configuration as specified: its step count, its decision interval, statistics on the
    decision steps, and for cfg3 the width change of 10 % of the tensors on every decision step
    (alternately by stq_repack between steps and fused into the step).  The last three are the other
    models of Table 1 under fp16 training: loss-scaled fp16 gradients and an fp16 working copy."""
    import harness as H
    import oracle
    _need(gib)
    w = W.config(name.split(":")[0])
    if name.endswith(":pl"):      # the same configuration with the piecewise-linear variant of the v quantizer
        from dataclasses import replace
        w = replace(w, v_log="pl")
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv)
    so = H.SampledOracle(job, per_tensor=4, seed=1)
    so.compare(0.0, f"{name} init")
    decisions = 0
    got = None
    for t in range(1, w.steps + 1):
        job.draw_grads(t)
        dec = t % w.decision_interval == 0 or t < 5
        new_bits = None
        if dec and w.churn > 0 and t >= 5:
            nbm, nbv, _ = W.churn_bits(w, job.bits_m, job.bits_v, decisions)
            decisions += 1
            if decisions % 2 == 0:
                new_bits = (nbm, nbv)
            else:
                job.repack((nbm, nbv))
                so.repack((nbm, nbv))
        so.step(t, new_bits=new_bits)
        job.step(t, stats=dec, new_bits=new_bits)
        so.compare(1e-6 * t if t <= 10 else 1e-4, f"{name} t={t}")
        if dec:
            got = job.layer_stats()
    for i, g in enumerate(job.grads):     # statistics of the last decision step (the last step of every config)
        if g.numel() <= (1 << 21):
            want = oracle.grad_stats(H.to_np(g.float() / w.loss_scale if w.loss_scale > 0 else g))
        else:
            g64 = g.double() * (1.0 / w.loss_scale if w.loss_scale > 0 else 1.0)
            want = np.array([g64.sum().item(), g64.abs().sum().item(), (g64 * g64).sum().item(), g.numel()])
        H.assert_stats_close(got[i:i + 1], want[None, :], f"{name} stats tensor {i}")
    # memory accounting of the problem statement: sum over layers of N_l * (b_m + b_v) bits (+ scales)
    bits = sum(n * (int(a) + int(b)) for n, a, b in zip(w.numels, job.bits_m, job.bits_v))
    code_bytes = sum(s.m_codes.numel() + s.v_codes.numel() for s in job.states)
    assert bits / 8 <= code_bytes <= bits / 8 + 32 * job.L
    assert job.state_bytes() < 0.25 * 8 * w.total_params     # far below the fp32 states


@pytest.mark.parametrize("name,gib,full_steps", [("cfg2", 8, None), ("cfg3", 6, None), ("cfg4", 30, 3), ("cfg5", 60, 3),
                                                 ("cfg2:sr", 8, 3), ("cfg3:ts", 6, 3),
                                                 ("cfg2:tile", 8, 12), ("cfg3:tile", 6, 40), ("cfg5:tile", 60, 2)])
def test_full_size_every_element(name, gib, full_steps):
    """Whole buffers against the oracle: every code byte, every scale, every parameter, on every step
    run (all of them for cfg2 and cfg3; steps 1-3 for cfg4 and cfg5, which are decision steps with fused
    statistics).  cfg3 changes the widths of 10 % of its tensors on every decision step from t = 5 on,
    alternately by stq_repack and inside the step.  The ":sr" and ":ts" cases run the first steps of a
    configuration with the stochastic-rounding or the two-scale code of the second moment.  The ":tile" cases
    keep every tensor in storage padded with zeros to whole tiles and give the library the padded lengths (a
    step is then one launch): the real elements' codes, scales and parameters are those of the oracle's run on
    the unpadded tensors."""
    import harness as H
    _need(gib)
    w = W.config(name.split(":")[0])
    tile = name.endswith(":tile")
    if ":" in name and not tile:  # the same configuration with another code of the second moment (its fused bodies)
        from dataclasses import replace
        w = replace(w, v_log=name.split(":")[1])
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv, tile_padded=tile)
    fo = H.FullOracle(job)
    fo.compare(0.0, f"{name} init")
    decisions = 0
    for t in range(1, (full_steps or w.steps) + 1):
        job.draw_grads(t)
        dec = t % w.decision_interval == 0 or t < 5
        new_bits = None
        if dec and w.churn > 0 and t >= 5:
            nbm, nbv, _ = W.churn_bits(w, job.bits_m, job.bits_v, decisions)
            decisions += 1
            if decisions % 2 == 0:
                new_bits = (nbm, nbv)
            else:
                job.repack((nbm, nbv))
                fo.repack((nbm, nbv))
        st_o = fo.step(t, new_bits=new_bits, want_stats=dec)
        n0 = job.handle.launch_count
        job.step(t, stats=dec, new_bits=new_bits)
        if tile and not dec:
            assert job.handle.launch_count - n0 == 1, "a plain step over tile-padded storage is one launch"
        fo.compare(1e-6 * t if t <= 10 else 1e-4, f"{name} t={t}")
        if dec:
            H.assert_stats_close(job.layer_stats(), st_o, f"{name} t={t}")
    assert job.handle.launch_count > 0


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


def _whole(t):
    """All bytes of the allocation a host tensor lives in."""
    return torch.empty(0, dtype=torch.uint8).set_(t.untyped_storage())


@pytest.mark.parametrize("flat", [True, False])
@pytest.mark.parametrize("stats", [False, True])
def test_host_buffer_step_matches_device_step(flat, stats):
    """stq_step_host (host pointers, copies inside the call) against stq_step on device buffers, with
    the host buffers of each kind in one flat allocation (a chunk then travels as one copy per kind)
    and allocated one by one.  The padding between flat buffers comes back untouched."""
    from paper_2604_06836_b200 import stq
    w = W.scaled(W.config("cfg4"), W.small_gpt2(d=136, n_layer=2), steps=2)
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv)
    job.draw_grads(1)
    job.step(1)
    job.draw_grads(2)
    tbl, hstates, hp_, hg = job.host_table(flat=flat)
    wholes = [_whole(t) for t in (hstates[0].m_codes, hstates[0].v_codes, hstates[0].m_scales, hstates[0].v_scales)]
    if flat:       # a pattern in the padding between the buffers
        for wh, ts in zip(wholes, ([s.m_codes for s in hstates], [s.v_codes for s in hstates],
                                   [s.m_scales for s in hstates], [s.v_scales for s in hstates])):
            keep = [t.clone() for t in ts]
            wh.fill_(0xA5)
            for t, k in zip(ts, keep):
                t.copy_(k)
    before = [wh.clone() for wh in wholes]
    flags = stq.WITH_STATS if stats else 0
    h2d, d2h = job.handle.step_host(tbl, flags=flags, **job.hp(2))
    got_stats = job.layer_stats() if stats else None
    job._tbl = None
    job.step(2, stats=stats)
    torch.cuda.synchronize()
    assert h2d > 0 and d2h > 0
    assert torch.equal(hp_, job.param_flat.cpu())
    for hs, s in zip(hstates, job.states):
        assert torch.equal(hs.m_codes, s.m_codes.cpu()) and torch.equal(hs.v_codes, s.v_codes.cpu())
        assert torch.equal(hs.m_scales, s.m_scales.cpu()) and torch.equal(hs.v_scales, s.v_scales.cpu())
    if stats:
        np.testing.assert_array_equal(got_stats, job.layer_stats())
    if flat:
        for wh, b4, ts in zip(wholes, before, ([s.m_codes for s in hstates], [s.v_codes for s in hstates],
                                               [s.m_scales for s in hstates], [s.v_scales for s in hstates])):
            covered = torch.zeros(wh.numel(), dtype=torch.bool)
            base = wh.data_ptr()
            for t in ts:
                o = t.data_ptr() - base
                covered[o:o + t.numel() * t.element_size()] = True
            assert torch.equal(wh[~covered], b4[~covered])
            assert (wh[~covered] == 0xA5).all()


@pytest.mark.parametrize("v_log", ["sr", "ts"])
def test_host_buffer_step_with_the_other_codes_of_v(v_log):
    """The host-buffer call with the stochastic-rounding code (same random words: they are keyed on the row's
    sr_id and the element's place in its row, not on the chunk a row travels in) and with the two-scale code
    (twice the scale bytes)."""
    from dataclasses import replace
    w = replace(W.scaled(W.config("cfg4"), W.small_gpt2(d=136, n_layer=2), steps=2), v_log=v_log)
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv)
    job.draw_grads(1)
    job.step(1)
    job.draw_grads(2)
    tbl, hstates, hp_, hg = job.host_table(flat=True)
    h2d, d2h = job.handle.step_host(tbl, **job.hp(2))
    job._tbl = None
    job.step(2)
    torch.cuda.synchronize()
    assert torch.equal(hp_, job.param_flat.cpu())
    for hs, s in zip(hstates, job.states):
        assert torch.equal(hs.m_codes, s.m_codes.cpu()) and torch.equal(hs.v_codes, s.v_codes.cpu())
        assert torch.equal(hs.m_scales, s.m_scales.cpu()) and torch.equal(hs.v_scales, s.v_scales.cpu())
        if v_log == "ts":
            assert hs.v_scales.numel() == 2 * hs.m_scales.numel()


def test_host_buffer_step_with_a_width_change_and_mixed_layouts():
    """Flat parameters and gradients, states allocated one by one, and new widths written to separate
    host buffers: the run path and the one-by-one path serve the same call."""
    from paper_2604_06836_b200 import stq
    w = W.scaled(W.config("cfg2"), W.small_gpt2(d=72, n_layer=1, vocab=301, ctx=16), steps=2)
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv)
    job.draw_grads(1)
    job.step(1)
    job.draw_grads(2)
    _, hstates, hp_, hg = job.host_table(flat=False)
    from dataclasses import replace
    nbm, nbv, _ = W.churn_bits(replace(w, churn=0.5), job.bits_m, job.bits_v, 0)
    new_h = [stq.QState(torch.zeros(stq.codes_bytes(n, int(a)), dtype=torch.uint8).pin_memory(),
                        torch.zeros(max(1, (n + w.block - 1) // w.block), dtype=torch.float32).pin_memory(), int(a),
                        torch.zeros(stq.codes_bytes(n, int(b)), dtype=torch.uint8).pin_memory(),
                        torch.zeros(max(1, (n + w.block - 1) // w.block), dtype=torch.float32).pin_memory(), int(b))
             for n, a, b in zip(job.numels, nbm, nbv)]
    rows = [stq.make_row(n, job.block, hstates[i], new_h[i], hp_[o:o + n], hg[o:o + n], job.wd[i])
            for i, (n, o) in enumerate(zip(job.numels, job.offsets))]
    job.handle.step_host(stq.table(rows), **job.hp(2))
    job._tbl = None
    job.step(2, new_bits=(nbm, nbv))
    torch.cuda.synchronize()
    assert torch.equal(hp_, job.param_flat.cpu())
    for hs, s in zip(new_h, job.states):
        assert torch.equal(hs.m_codes, s.m_codes.cpu()) and torch.equal(hs.v_codes, s.v_codes.cpu())
        nb = s.m_scales.numel()
        assert torch.equal(hs.m_scales[:nb], s.m_scales.cpu()) and torch.equal(hs.v_scales[:nb], s.v_scales.cpu())


def test_a_wait_that_runs_out_is_reported_and_the_context_survives():
    """Every wait in the kernels is bounded; when one runs out the kernel raises a flag and returns.
    The self-test takes that path with a 0.1 ms limit on a barrier nothing completes."""
    from paper_2604_06836_b200 import stq
    h = stq.Handle()
    h.device_status()                                   # clean
    h.selftest_wait_timeout()
    with pytest.raises(stq.StqError) as ei:
        h.device_status()
    assert ei.value.code == -11
    h.close()
    # the context is alive and a fresh handle works
    w = W.scaled(W.config("cfg2"), W.small_gpt2(d=72, n_layer=1, vocab=200), steps=1)
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv)
    job.draw_grads(1)
    job.step(1)
    job.handle.device_status()
    assert torch.isfinite(job.param_flat).all()


def test_nothing_is_written_outside_the_callers_buffers():
    """Every buffer sits between guard regions filled with a pattern; after init, steps with and
    without a width change, and a re-pack, the guards are intact (ragged sizes, all widths)."""
    from paper_2604_06836_b200 import stq
    dev = "cuda"
    G = 256   # guard bytes on each side
    h = stq.Handle()

    def guarded(nbytes):
        buf = torch.full((nbytes + 2 * G,), 0xA5, dtype=torch.uint8, device=dev)
        return buf, buf[G:G + nbytes]

    def intact(buf, nbytes):
        return bool((buf[:G] == 0xA5).all() and (buf[G + nbytes:] == 0xA5).all())

    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8)
    for n in (1, 129, 1000, 4097, 12289 + 77):
        for (bm, bv, bm2, bv2) in [(3, 3, 3, 3), (2, 16, 8, 4), (8, 4, 32, 3), (16, 2, 2, 32)]:
            bufs = {}
            def mk(name, nbytes):
                bufs[name] = guarded(nbytes) + (nbytes,)
                return bufs[name][1]
            p = mk("p", _r16(4 * n)).view(torch.float32)[:n]
            g = mk("g", _r16(4 * n)).view(torch.float32)[:n]
            p.normal_(0, 0.02); g.normal_(0, 1e-3)
            sb = stq.scales_bytes(n, 128)
            def state(tag, a, b):
                return stq.QState(mk(tag + "mc", stq.codes_bytes(n, a)), mk(tag + "ms", _r16(sb)).view(torch.float32)[:sb // 4], a,
                                  mk(tag + "vc", stq.codes_bytes(n, b)), mk(tag + "vs", _r16(sb)).view(torch.float32)[:sb // 4], b)
            s1, s2, s3 = state("a", bm, bv), state("b", bm2, bv2), state("c", bm, bv)
            h.init_state(stq.table([stq.make_row(n, 128, None, s1)]))
            h.step(stq.table([stq.make_row(n, 128, s1, s1, p, g, 0.01)]), t=1, **hp)            # in place
            h.step(stq.table([stq.make_row(n, 128, s1, s2, p, g, 0.01)]), t=2, **hp)            # width change in the step
            h.repack(stq.table([stq.make_row(n, 128, s2, s3)]))                                  # and back by re-pack
            h.device_status()
            for name, (buf, _, nbytes) in bufs.items():
                assert intact(buf, nbytes), (n, bm, bv, bm2, bv2, name)


def _r16(x):
    return (x + 15) // 16 * 16


def test_one_tensor_beyond_two_to_the_31_elements():
    """Element indices past 2^31 and byte offsets past 2^33: one tensor of 2^31 + 20,813 elements (fast
    tiles plus a ragged tail in the generic kernel), checked on sampled blocks (first, last, tail, random)."""
    import harness as H
    _need(40)
    n = (1 << 31) + 4096 * 5 + 333
    w = W.Workload("one-tensor-2^31", (("w", (n,)),), 128, "bf16", "student_t", nu=3, scale_log10=(-3.0, -3.0),
                   bits_kind="fixed", bits_fixed=(4, 8), seed=11)
    job = Job(w, [4], [8])
    so = H.SampledOracle(job, per_tensor=12, seed=2)
    for t in (1, 2):
        job.draw_grads(t)
        so.step(t)
        job.step(t, stats=True)
        so.compare(1e-6 * t, f"2^31 t={t}")
        got = job.layer_stats()
        g = job.grads[0]
        want = np.zeros(4)
        for lo in range(0, n, 1 << 28):          # float64 sums, a slice at a time
            x = g[lo:lo + (1 << 28)].double()
            want += np.array([x.sum().item(), x.abs().sum().item(), (x * x).sum().item(), x.numel()])
        H.assert_stats_close(got, want[None, :], f"2^31 t={t}")
    # the gradient-only pass over the same gradients
    job.handle.grad_stats(job.table(), job.grad_dtype)
    H.assert_stats_close(job.layer_stats(), want[None, :], "2^31 statistics alone")


def test_one_tensor_beyond_two_to_the_32_elements():
    """The largest class of tensor the table accepts on one GPU: more than 2^32 elements, which the main
    kernel leaves to the generic one (its tile counters are 32-bit); 64-bit element indices throughout."""
    import harness as H
    _need(90)
    n = (1 << 32) + 4096 * 3 + 77
    w = W.Workload("one-tensor-2^32", (("w", (n,)),), 256, "bf16", "normal", scale_log10=(-3.0, -3.0),
                   bits_kind="fixed", bits_fixed=(3, 4), seed=12)
    job = Job(w, [3], [4])
    so = H.SampledOracle(job, per_tensor=12, seed=3)
    job.draw_grads(1)
    so.step(1)
    job.step(1, stats=True)
    so.compare(1e-6, "2^32 t=1")
    got = job.layer_stats()
    assert got[0, 3] == n
    g = job.grads[0]
    want = np.zeros(4)
    for lo in range(0, n, 1 << 28):
        x = g[lo:lo + (1 << 28)].double()
        want += np.array([x.sum().item(), x.abs().sum().item(), (x * x).sum().item(), x.numel()])
    H.assert_stats_close(got, want[None, :], "2^32")
    job.handle.grad_stats(job.table(), job.grad_dtype)
    H.assert_stats_close(job.layer_stats(), want[None, :], "2^32 statistics alone")


def test_full_size_runs_are_identical_bit_for_bit():
    """The tile order a CTA sees depends on dynamic scheduling (atomic chunk counters), the results must
    not: two runs of cfg2 (30 steps, statistics every 10th, a width change on the way) end in the same
    parameters, codes, scales and statistics."""
    _need(6)
    w = W.config("cfg2")
    bm, bv, _ = W.draw_bits(w)

    def run():
        job = Job(w, bm, bv)
        stats = []
        for t in range(1, 31):
            job.draw_grads(t)
            new_bits = None
            if t == 20:
                new_bits = W.churn_bits(__import__("dataclasses").replace(w, churn=0.2), job.bits_m, job.bits_v, 0)[:2]
            job.step(t, stats=(t % 10 == 0), new_bits=new_bits)
            if t % 10 == 0:
                stats.append(job.layer_stats())
        job.handle.device_status()
        return job, stats

    a, sa = run()
    b, sb = run()
    assert torch.equal(a.param_flat, b.param_flat)
    for x, y in zip(a.states, b.states):
        assert x.bits_m == y.bits_m and x.bits_v == y.bits_v
        assert torch.equal(x.m_codes, y.m_codes) and torch.equal(x.v_codes, y.v_codes)
        assert torch.equal(x.m_scales, y.m_scales) and torch.equal(x.v_scales, y.v_scales)
    for x, y in zip(sa, sb):
        np.testing.assert_array_equal(x, y)

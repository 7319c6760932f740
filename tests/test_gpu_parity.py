"""Parity of the CUDA path with the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2604_06836_b200 import stq, workloads as W   # noqa: E402
from paper_2604_06836_b200.runner import Job             # noqa: E402

REL_1STEP = 1e-6     # parameters after one step
REL_100 = 1e-4       # parameters after 100 steps


@pytest.fixture(scope="module")
def H():
    import harness
    return harness


def _single(n, block, gdt, seed=0):
    return W.Workload(f"single-{n}", (("w", (n,)),), block, gdt, "student_t", nu=4,
                      scale_log10=(-3.0, -3.0), bits_kind="fixed", seed=seed)


@pytest.mark.parametrize("gdt", ["fp32", "bf16"])
@pytest.mark.parametrize("block", [128, 256, 512])
@pytest.mark.parametrize("bm", [2, 3, 4, 8, 16])
@pytest.mark.parametrize("bv", [2, 3, 4, 8, 16])
def test_every_width_pair_three_steps(H, O, bm, bv, block, gdt):
    n = 4096 * 3 + 128 * 5 + 52          # several tiles, a partial tile, a ragged last block
    w = _single(n, block, gdt, seed=bm * 100 + bv)
    job = Job(w, [bm], [bv])
    oj = H.OracleJob(job)
    H.compare_job(job, oj, 0.0, "init")
    for t in (1, 2, 3):
        job.draw_grads(t)
        oj.step([H.to_np(g) for g in job.grads], t)
        job.step(t)
        H.compare_job(job, oj, REL_1STEP * t, f"t={t}")


@pytest.mark.parametrize("n", [1, 2, 3, 5, 127, 128, 129, 255, 257, 1000, 4095, 4096, 4097, 8191, 12289])
@pytest.mark.parametrize("bits", [(3, 3), (8, 4), (16, 2), (2, 16)])
def test_ragged_sizes(H, O, n, bits):
    for block, gdt in ((128, "fp32"), (256, "bf16")):
        w = _single(n, block, gdt, seed=n)
        job = Job(w, [bits[0]], [bits[1]])
        oj = H.OracleJob(job)
        for t in (1, 2):
            job.draw_grads(t)
            st = oj.step([H.to_np(g) for g in job.grads], t, want_stats=True)
            job.step(t, stats=True)
            H.compare_job(job, oj, REL_1STEP * t, f"n={n} t={t}")
            H.assert_stats_close(job.layer_stats(), st, f"n={n}")


def test_states_at_32_bits_and_mixed(H, O):
    """Raw fp32 states (the paper's 32-bit candidate) and tables mixing 32-bit and packed tensors."""
    shapes = [("a", (5000,)), ("b", (4096,)), ("c", (777,)), ("d", (9000,))]
    w = W.Workload("mixed32", tuple(shapes), 128, "fp32", "student_t", nu=4, scale_log10=(-4.0, -2.0), seed=11)
    job = Job(w, [32, 8, 32, 4], [32, 32, 3, 4])
    oj = H.OracleJob(job)
    for t in range(1, 6):
        job.draw_grads(t)
        oj.step([H.to_np(g) for g in job.grads], t)
        job.step(t)
        H.compare_job(job, oj, REL_1STEP * t, f"t={t}")


def test_cfg1_single_tensor_warmup_then_m8_v4(H, O):
    """1,048,576 parameters: ten warm-up steps with fp32 states, quantize to m8/v4, measured step 11 with stats."""
    w = W.config("cfg1")
    job = Job(w, [32], [32])
    oj = H.OracleJob(job)
    for t in range(1, w.warmup_fp32_steps + 1):
        job.draw_grads(t)
        oj.step([H.to_np(g) for g in job.grads], t)
        job.step(t)
    H.compare_job(job, oj, REL_1STEP * 10, "warm-up")   # fp32 moments are bit-exact, theta has rounded 10 times
    job.repack(([8], [4]))
    oj.repack(([8], [4]))
    H.compare_job(job, oj, REL_1STEP * 10, "quantized")
    t = w.warmup_fp32_steps + 1
    job.draw_grads(0)
    before = [th.copy() for th in oj.theta]
    st = oj.step([H.to_np(g) for g in job.grads], t, want_stats=True)
    # measured step alone: start the GPU from the oracle's parameters so only one step's rounding shows
    job.params[0].copy_(torch.from_numpy(before[0]).cuda())
    job.step(t, stats=True)
    H.compare_job(job, oj, REL_1STEP, "measured step")
    H.assert_stats_close(job.layer_stats(), st, "cfg1")


def _run_config(H, w, steps, churn_in_step=True):
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv)
    oj = H.OracleJob(job)
    pol_g = stq.Policy(alpha=0.1, tau=100.0, eps_stat=1e-8, interval=w.decision_interval)
    import oracle
    pol_o = oracle.new_policy(0.1, 100.0, 1e-8)
    decision = 0
    for t in range(1, steps + 1):
        job.draw_grads(t)
        grads = [H.to_np(g) for g in job.grads]
        dec = pol_g.is_decision_step(t)
        assert dec == oracle.is_decision_step(t, w.decision_interval)
        new_bits = None
        if dec and w.churn > 0 and t >= 5:
            nbm, nbv, _ = W.churn_bits(w, job.bits_m, job.bits_v, decision)
            decision += 1
            if churn_in_step and decision % 2 == 0:
                new_bits = (nbm, nbv)          # width change fused into the step
            else:
                job.repack((nbm, nbv))         # width change between steps
                oj.repack((nbm, nbv))
        st_o = oj.step(grads, t, want_stats=dec, new_bits=new_bits)
        job.step(t, stats=dec, new_bits=new_bits)
        rel = REL_1STEP * max(1, t) if t <= 10 else REL_100
        H.compare_job(job, oj, rel, f"{w.name} t={t}")
        if dec:
            st_g = job.layer_stats()
            H.assert_stats_close(st_g, st_o, f"{w.name} t={t}")
            # the paper's policy runs in shadow on both sides, on the GPU's statistics
            bg, sg = pol_g.decide(st_g, t)
            bo, so = oracle.decide(pol_o, st_g, t)
            assert (bg == bo).all()
            np.testing.assert_allclose(sg, so, rtol=1e-12, atol=1e-12)
    return job, oj


def test_small_gpt2_100_steps_k10(H, O):
    w = W.scaled(W.config("cfg2"), W.small_gpt2(), steps=100)
    _run_config(H, w, 100)


def test_small_vit_100_steps_k20_with_width_churn(H, O):
    w = W.scaled(W.config("cfg3"), W.small_vit(), steps=100)
    _run_config(H, w, 100)


def test_small_gpt2_bf16_m48_v348(H, O):
    w = W.scaled(W.config("cfg4"), W.small_gpt2(d=136, n_layer=3), steps=50)
    _run_config(H, w, 50)


def test_small_gpt2_xl_recipe(H, O):
    w = W.scaled(W.config("cfg5"), W.small_gpt2(d=100, n_layer=4, vocab=523), steps=20)
    _run_config(H, w, 20)


def test_l2_mode_and_per_tensor_weight_decay(H, O):
    shapes = [("a", (3000,)), ("b", (513,))]
    w = W.Workload("l2", tuple(shapes), 128, "fp32", "normal", scale_log10=(-3.0, -3.0), seed=5)
    job = Job(w, [8, 4], [4, 8])
    job.wd = [0.1, 0.0]
    job._tbl = None
    oj = H.OracleJob(job)
    for t in (1, 2, 3):
        job.draw_grads(t)
        oj.step([H.to_np(g) for g in job.grads], t, decoupled_wd=False)
        job.handle.step(job.table(), decoupled_wd=False, **job.hp(t))
        H.compare_job(job, oj, REL_1STEP * t, f"l2 t={t}")


def test_grad_stats_only_pass(H, O):
    import oracle
    w = W.scaled(W.config("cfg4"), W.small_gpt2(d=136, n_layer=1), steps=1)
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv)
    job.draw_grads(1)
    job.handle.grad_stats(job.table(), job.grad_dtype)
    got = job.layer_stats()
    want = np.stack([oracle.grad_stats(H.to_np(g)) for g in job.grads])
    H.assert_stats_close(got, want, "stats-only")
    job._tbl = None
    job.step(1)     # the step table is rebuilt after a stats-only table


def test_run_to_run_identical(H, O):
    w = W.scaled(W.config("cfg2"), W.small_gpt2(), steps=3)
    outs = []
    for _ in range(2):
        bm, bv, _ = W.draw_bits(w)
        job = Job(w, bm, bv)
        for t in (1, 2, 3):
            job.draw_grads(t)
            job.step(t, stats=True)
        st = job.layer_stats()
        outs.append((torch.cat([p.clone() for p in job.params]).cpu(), st,
                     torch.cat([s.m_codes for s in job.states] + [s.v_codes for s in job.states]).cpu()))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][2], outs[1][2])
    assert (outs[0][1] == outs[1][1]).all()


def test_algorithm1_order_with_the_paper_policy_driving_the_widths(H, O):
    """Algorithm 1 as printed: on decision steps the statistics of the fresh gradients are taken first,
    the policy maps them to widths in {4, 8, 16, 32}, and the same step already writes the states at the
    new widths (every layer starts at 16 bits)."""
    import oracle
    w = W.scaled(W.config("cfg2"), W.small_gpt2(d=136, n_layer=2, vocab=300), steps=24)
    L = len(w.shapes)
    job = Job(w, [16] * L, [16] * L)
    oj = H.OracleJob(job)
    U = 6
    pol_g = stq.Policy(alpha=0.1, tau=8.0, eps_stat=1e-8, interval=U)
    pol_o = oracle.new_policy(0.1, 8.0, 1e-8)
    seen = set()
    for t in range(1, 25):
        job.draw_grads(t)
        grads = [H.to_np(g) for g in job.grads]
        new_bits = None
        if pol_g.is_decision_step(t):
            job.handle.grad_stats(job.table(), job.grad_dtype)
            st_g = job.layer_stats()
            job._tbl = None
            st_o = np.stack([oracle.grad_stats(g) for g in grads])
            H.assert_stats_close(st_g, st_o, f"t={t}")
            bg, _ = pol_g.decide(st_g, t)
            bo, _ = oracle.decide(pol_o, st_g, t)
            assert (bg == bo).all() and set(bg.tolist()) <= {4, 8, 16, 32}
            new_bits = (bg, bg)                      # Algorithm 1: one width per layer for both states
            seen |= set(bg.tolist())
        oj.step(grads, t, new_bits=new_bits)
        job.step(t, new_bits=new_bits)
        H.compare_job(job, oj, REL_1STEP * t if t <= 10 else REL_100, f"t={t}")
    assert len(seen) >= 2          # the policy did move layers between widths


@pytest.mark.parametrize("gdt", [torch.float16, torch.bfloat16, torch.float32])
def test_loss_scaled_gradients_skip_flag_and_low_precision_copy(H, O, gdt):
    """Mixed-precision training plumbing fused into the step: gradients arrive multiplied by the loss
    scale (fp16 here, as the paper trains), are brought back by *inv_grad_scale before anything else,
    found_inf skips the step, and the updated parameters are also written as a bf16 / fp16 copy."""
    import oracle
    shapes = [("a", (4096 * 2 + 700,)), ("b", (333,)), ("c", (4096,))]
    w = W.Workload("amp", tuple(shapes), 128, "fp32", "student_t", nu=4, scale_log10=(-4.0, -3.0), seed=21)
    S = 1024.0
    job = Job(w, [8, 4, 3], [4, 8, 2])
    oj = H.OracleJob(job)
    inv = torch.tensor([1.0 / S], dtype=torch.float32, device="cuda")
    flag = torch.zeros(1, dtype=torch.float32, device="cuda")
    lp_dt = torch.float16 if gdt == torch.float16 else torch.bfloat16
    lps = [torch.zeros(n, dtype=lp_dt, device="cuda") for n in job.numels]
    grads = [torch.zeros(n, dtype=gdt, device="cuda") for n in job.numels]
    rows = lambda: stq.table([stq.make_row(n, job.block, job.states[i], job.states[i], job.params[i], grads[i],
                                            job.wd[i], lps[i]) for i, n in enumerate(job.numels)])
    for t in (1, 2, 3, 4):
        job.draw_grads(t)
        for i in range(job.L):
            grads[i].copy_((job.grads[i] * S).to(gdt))
        skip = (t == 3)
        flag.fill_(1.0 if skip else 0.0)
        before = [p.clone() for p in job.params]
        codes_before = [s.m_codes.clone() for s in job.states]
        st_o = oj.step([H.to_np(g) for g in grads], t, want_stats=True, fp16_grad=(gdt == torch.float16),
                       inv_grad_scale=1.0 / S, found_inf=skip)
        job.handle.step(rows(), flags=stq.WITH_STATS,
                        **{**job.hp(t), "grad_dtype": stq.grad_dtype_of(grads[0]), "inv_grad_scale": inv,
                           "found_inf": flag})
        H.compare_job(job, oj, REL_1STEP * t, f"{gdt} t={t}")
        if skip:
            assert all(torch.equal(a, b) for a, b in zip(before, job.params))
            assert all(torch.equal(a, s.m_codes) for a, s in zip(codes_before, job.states))
            # the skipped step produced no sums: asking for them is a call-order error, not stale numbers
            flag.fill_(0.0)                        # (the flag was read when the step ran; reusing it changes nothing)
            with pytest.raises(stq.StqError) as err:
                job.handle.layer_stats(job.L)
            assert err.value.code == stq.E_STATE
        else:
            H.assert_stats_close(job.handle.layer_stats(job.L), st_o, f"{gdt} t={t}")
            for i in range(job.L):
                # the copy is exactly the nearest-even rounding of the parameters the kernel wrote
                assert torch.equal(lps[i], job.params[i].to(lp_dt)), (t, i)
                want = oracle.round_lp(oj.theta[i], "fp16" if lp_dt == torch.float16 else "bf16")
                got = H.to_np(lps[i])
                assert (np.abs(got.astype(np.int32) - want.astype(np.int32)) <= 1).all()   # a last-bit tie at most


def test_extreme_but_finite_values(H, O):
    """Zero blocks, denormal gradients (the tiny-scale rule), huge gradients, one outlier per block,
    alternating signs: codes and scales stay bit-exact and nothing faults."""
    n = 4096 * 2 + 128 * 3
    w = W.Workload("extreme", (("a", (n,)), ("b", (n,)), ("c", (n,))), 128, "fp32", "normal",
                   scale_log10=(-3.0, -3.0), seed=31)
    job = Job(w, [8, 3, 16], [4, 8, 2])
    oj = H.OracleJob(job)
    g = torch.Generator(device="cuda").manual_seed(3)
    for t in range(1, 6):
        for i in range(3):
            x = torch.randn(n, generator=g, device="cuda") * 1e-3
            blk = x.view(-1, 128)
            blk[0::7] = 0.0                                    # all-zero blocks
            blk[1::7] *= 1e-42                                 # denormal gradients
            blk[2::7] *= 1e-25                                 # v below the tiny-scale rule, m above it
            blk[3::7] *= 1e16                                  # large: v up to ~1e23
            blk[4::7, 5] = 3e3                                 # one outlier dwarfs its block
            blk[5::7] = blk[5::7].abs() * (1 - 2 * (torch.arange(128, device="cuda") % 2))   # +-+-
            job.grads[i].copy_(x)
        oj.step([H.to_np(gr) for gr in job.grads], t, want_stats=False)
        job.step(t)
        H.compare_job(job, oj, REL_1STEP * t, f"extreme t={t}")


def test_non_finite_gradients_do_not_fault_or_leak_into_other_blocks(H, O):
    """Inf / NaN gradients are outside the contract (use found_inf): the affected blocks hold garbage,
    but the kernel neither faults nor disturbs any other block."""
    n = 4096 + 512
    w = W.Workload("nonfinite", (("a", (n,)),), 128, "fp32", "normal", scale_log10=(-3.0, -3.0), seed=32)
    job = Job(w, [4], [4])
    oj = H.OracleJob(job)
    job.draw_grads(1)
    bad_blocks = [3, 17, 35]
    for b, val in zip(bad_blocks, (float("inf"), float("nan"), -float("inf"))):
        job.grads[0][b * 128 + 7] = val
    good = np.ones(n, bool)
    for b in bad_blocks:
        good[b * 128:(b + 1) * 128] = False
    gnp = H.to_np(job.grads[0])
    gnp_clean = np.where(good, gnp, 0).astype(np.float32)
    oj.step([gnp_clean], 1)
    job.step(1)
    job.handle.device_status()
    th = H.to_np(job.params[0])
    assert np.allclose(th[good], oj.theta[0][good], rtol=2e-6, atol=1e-9)
    gm = H.to_np(job.states[0].m_codes)
    om = oj.states[0].m_codes
    keep = np.repeat(good.reshape(-1, 128)[:, 0], 64)       # 4-bit codes: 64 bytes per block
    assert (gm[:keep.size][keep] == om[:keep.size][keep]).all()


@pytest.mark.parametrize("bits", [(4, 4), (3, 8), (8, 3), (16, 2)])
def test_element_ranges_of_a_tensor_step_like_the_whole_tensor(H, O, bits):
    """A sharded optimizer hands each rank ranges of a tensor cut on tile boundaries: stepping the
    ranges as rows of their own (here: two handles, one after the other) writes the same bits as
    stepping the whole tensor, and the per-layer sums of the ranges add up to the tensor's.  Each
    rank's range is also held against the oracle's run of exactly that range (its own parameters,
    gradients and zero-initialised state), codes and scales bit for bit."""
    import oracle
    from paper_2604_06836_b200 import multi, stq
    bm, bv = bits
    n, block, dev = 5 * 4096 + 777, 128, "cuda"
    g0 = torch.Generator(device=dev).manual_seed(5)
    theta = torch.empty(n, device=dev).normal_(0, 0.02, generator=g0)
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, grad_dtype=stq.GRAD_BF16)
    cuts = [r for sh in multi.partition([n], 2) for r in sh]
    assert len(cuts) == 2 and cuts[0][2] == cuts[1][1]

    def view(st, lo, hi):     # the range's slice of a whole-tensor state (no copy: same device memory)
        return stq.QState(st.m_codes[lo * bm // 8:], st.m_scales[lo // block:], bm,
                          st.v_codes[lo * bv // 8:], st.v_scales[lo // block:], bv)

    whole_p, split_p = theta.clone(), theta.clone()
    whole_s, split_s = stq.alloc_state(n, block, bm, bv, dev), stq.alloc_state(n, block, bm, bv, dev)
    h_whole, h_a, h_b = stq.Handle(), stq.Handle(), stq.Handle()
    h_whole.init_state(stq.table([stq.make_row(n, block, None, whole_s)]))
    for h, (_, lo, hi) in zip((h_a, h_b), cuts):
        h.init_state(stq.table([stq.make_row(hi - lo, block, None, view(split_s, lo, hi))]))
    o_theta = [H.to_np(theta[lo:hi]) for _, lo, hi in cuts]                     # the oracle's ranks
    o_state = [oracle.new_state(hi - lo, block, bm, bv) for _, lo, hi in cuts]
    for t in (1, 2, 3):
        g = (torch.empty(n, device=dev).normal_(0, 1e-3, generator=g0)).to(torch.bfloat16)
        h_whole.step(stq.table([stq.make_row(n, block, whole_s, whole_s, whole_p, g, 0.01)]), t=t,
                     flags=stq.WITH_STATS, **hp)
        total = np.zeros(4)
        for h, (_, lo, hi) in zip((h_a, h_b), cuts):
            v = view(split_s, lo, hi)
            h.step(stq.table([stq.make_row(hi - lo, block, v, v, split_p[lo:hi], g[lo:hi], 0.01)]), t=t,
                   flags=stq.WITH_STATS, **hp)
            got = h.layer_stats(1)
            total += got[0]
            k = 0 if lo == 0 else 1
            o_state[k], st_o = oracle.step(o_theta[k], H.to_np(g[lo:hi]), o_state[k], block, lr=1e-3, beta1=0.9,
                                           beta2=0.999, eps=1e-8, weight_decay=0.01, t=t, want_stats=True)
            mine = stq.QState(v.m_codes[:o_state[k].m_codes.size], v.m_scales[:o_state[k].m_scales.size], bm,
                              v.v_codes[:o_state[k].v_codes.size], v.v_scales[:o_state[k].v_scales.size], bv)
            H.assert_states_equal(mine, o_state[k], f"rank {k} t={t}")
            H.assert_theta_close(split_p[lo:hi], o_theta[k], REL_1STEP * t, f"rank {k} t={t}",
                                 upd=np.abs(o_theta[k]) + 2e-3)
            H.assert_stats_close(got, st_o[None, :], f"rank {k} t={t}")
        want = h_whole.layer_stats(1)[0]
        assert torch.equal(whole_p, split_p)
        for a, b in ((whole_s.m_codes, split_s.m_codes), (whole_s.v_codes, split_s.v_codes),
                     (whole_s.m_scales, split_s.m_scales), (whole_s.v_scales, split_s.v_scales)):
            assert torch.equal(a, b)
        assert total[3] == want[3] == n
        np.testing.assert_allclose(total[:3], want[:3], rtol=1e-6, atol=1e-12)


# ---- the piecewise-linear variant of the v quantizer -----------------------------------------------------
@pytest.mark.parametrize("gdt", ["fp32", "bf16"])
@pytest.mark.parametrize("block", [128, 256, 512])
@pytest.mark.parametrize("bm", [2, 3, 4, 8, 16])
@pytest.mark.parametrize("bv", [8, 16])
def test_pl_variant_every_width_pair(H, O, bm, bv, block, gdt):
    from dataclasses import replace
    n = 4096 * 3 + 128 * 5 + 52
    w = replace(_single(n, block, gdt, seed=bm * 100 + bv), v_log="pl")
    job = Job(w, [bm], [bv])
    oj = H.OracleJob(job)
    H.compare_job(job, oj, 0.0, "init")
    for t in (1, 2, 3):
        job.draw_grads(t)
        st = oj.step([H.to_np(g) for g in job.grads], t, want_stats=True)
        job.step(t, stats=True)
        H.compare_job(job, oj, REL_1STEP * t, f"pl t={t}")
        H.assert_stats_close(job.layer_stats(), st, "pl")


@pytest.mark.parametrize("n", [1, 5, 129, 1000, 4095, 4097, 12289])
def test_pl_variant_ragged_sizes(H, O, n):
    from dataclasses import replace
    for bits, block, gdt in (((8, 8), 128, "fp32"), ((3, 16), 256, "bf16")):
        w = replace(_single(n, block, gdt, seed=n), v_log="pl")
        job = Job(w, [bits[0]], [bits[1]])
        oj = H.OracleJob(job)
        for t in (1, 2):
            job.draw_grads(t)
            oj.step([H.to_np(g) for g in job.grads], t)
            job.step(t)
            H.compare_job(job, oj, REL_1STEP * t, f"pl n={n} t={t}")


def test_pl_variant_small_vit_with_width_churn(H, O):
    """100 steps with width changes between and inside steps (the octave widths are shared by both
    variants, so a change 4 -> 8 bits moves a state into the variant's code and back)."""
    from dataclasses import replace
    w = replace(W.scaled(W.config("cfg3"), W.small_vit(), steps=100), v_log="pl")
    _run_config(H, w, 100)


def test_pl_variant_small_gpt2_xl_recipe_bf16(H, O):
    from dataclasses import replace
    w = replace(W.scaled(W.config("cfg5"), W.small_gpt2(d=100, n_layer=4, vocab=523), steps=20), v_log="pl")
    _run_config(H, w, 20)


def test_pl_variant_extreme_values_and_mixed_tables(H, O):
    """Zero, denormal and huge blocks in the variant; and a table that mixes tensors of both variants."""
    n, block, dev = 4096 * 2 + 300, 128, "cuda"
    import oracle
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8)
    g = torch.zeros(n, device=dev)
    g[:128] = 0.0
    g[128:256] = 1e-30            # squares underflow: a zero block of v
    g[256:384] = 1e18             # v near the top of the fp32 range
    g[384:512] = torch.linspace(1e-12, 1e-3, 128, device=dev)
    g[4096:] = torch.empty(n - 4096, device=dev).normal_(0, 1e-3, generator=torch.Generator(device=dev).manual_seed(1))
    h = stq.Handle()
    states, thetas = [], []
    for v_log, bv in ((stq.VLOG_PL, 8), (stq.VLOG_POLY, 16), (stq.VLOG_PL, 16), (stq.VLOG_POLY, 8)):
        st = stq.alloc_state(n, block, 4, bv, dev, v_log)
        th = torch.full((n,), 0.01, device=dev)
        states.append(st)
        thetas.append(th)
    h.init_state(stq.table([stq.make_row(n, block, None, s) for s in states]))
    o_states = [oracle.new_state(n, block, s.bits_m, s.bits_v) for s in states]
    o_thetas = [H.to_np(t) for t in thetas]
    for t in (1, 2, 3):
        h.step(stq.table([stq.make_row(n, block, s, s, th, g, 0.01) for s, th in zip(states, thetas)]), t=t, **hp)
        h.device_status()
        for i, s in enumerate(states):
            o_states[i], _ = oracle.step(o_thetas[i], H.to_np(g), o_states[i], block, t=t, weight_decay=0.01,
                                         v_mode=oracle.LOG_PL if s.v_log == stq.VLOG_PL else oracle.LOG, **hp)
            H.assert_states_equal(s, o_states[i], f"mixed table row {i} t={t}")
            H.assert_theta_close(thetas[i], o_thetas[i], REL_1STEP * t, f"mixed table row {i} t={t}",
                                 upd=np.full(n, 0.01))
    # a bad variant id is refused before anything runs
    bad = stq.make_row(n, block, states[0], states[0], thetas[0], g, 0.01)
    bad.v_log = 7
    with pytest.raises(stq.StqError):
        h.step(stq.table([bad]), t=4, **hp)


@pytest.mark.parametrize("v_log", ["poly", "pl"])
def test_fp16_training_recipe_on_a_small_model(H, O, v_log):
    """Table 1's fp16 recipe (loss-scaled fp16 gradients, fp16 working copy) on a small GPT-2-shaped list,
    in both variants of the v code: the mixed-precision bodies of the step kernel against the oracle."""
    from dataclasses import replace
    w = replace(W.scaled(W.config("gpt2_medium"), W.small_gpt2(d=136, n_layer=2), steps=6), v_log=v_log)
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv)
    oj = H.OracleJob(job)
    for t in range(1, 7):
        job.draw_grads(t)
        st = oj.step([H.to_np(g) for g in job.grads], t, want_stats=True, fp16_grad=True,
                     inv_grad_scale=1.0 / w.loss_scale)
        job.step(t, stats=True)
        H.compare_job(job, oj, REL_1STEP * t, f"fp16 {v_log} t={t}")
        H.assert_stats_close(job.layer_stats(), st, f"fp16 {v_log} t={t}")
        for p, lp in zip(job.params, job.params_lp):
            assert torch.equal(lp, p.to(torch.float16))


def test_a_step_can_be_captured_into_a_cuda_graph(H, O):
    """A step over a table the handle has already seen enqueues only stream work (a counter reset, the
    kernels, the fork and join of the side stream), so it can be captured and replayed.  The scalars
    of the step (bias corrections, learning rate) are baked in at capture: a replay repeats step t."""
    w = W.scaled(W.config("cfg5"), W.small_gpt2(d=136, n_layer=2, vocab=777), steps=3)
    bm, bv, _ = W.draw_bits(w)

    def make():
        job = Job(w, bm, bv)
        job.draw_grads(1)
        job.step(1)
        return job

    eager, graphed = make(), make()
    for _ in range(3):
        eager.step(5)
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        graphed.handle.step(graphed.table(), **graphed.hp(5))      # step 1 of 3, and the table's first use
        s.synchronize()
        with torch.cuda.graph(g, stream=s):
            graphed.handle.step(graphed.table(), **graphed.hp(5))  # captured, not run
        g.replay()                                                  # steps 2 and 3
        g.replay()
        s.synchronize()
    graphed.handle.device_status()
    assert torch.equal(eager.param_flat, graphed.param_flat)
    for x, y in zip(eager.states, graphed.states):
        assert torch.equal(x.m_codes, y.m_codes) and torch.equal(x.v_codes, y.v_codes)
        assert torch.equal(x.m_scales, y.m_scales) and torch.equal(x.v_scales, y.v_scales)


def test_graph_replays_advance_with_a_step_count_on_the_device(H, O):
    """The step count and the learning rate may live on the device (hparams.step_dev / lr_dev): a step
    captured once then runs steps t, t+1, ... as the caller's counter advances inside the graph, with new
    gradients copied into the same buffers before every replay.  Codes and scales are those of eager
    steps; the parameters agree to rounding (the device forms lr / (1 - beta1^t) from a float32 lr)."""
    w = W.scaled(W.config("cfg2"), W.small_gpt2(d=136, n_layer=2, vocab=777), steps=8)
    bm, bv, _ = W.draw_bits(w)
    eager, graphed = Job(w, bm, bv), Job(w, bm, bv)
    oj = H.OracleJob(eager)
    step_dev = torch.zeros(1, dtype=torch.int64, device="cuda")
    lr_dev = torch.full((1,), w.lr, dtype=torch.float32, device="cuda")
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    hp = {**graphed.hp(1), "step_dev": step_dev, "lr_dev": lr_dev}
    with torch.cuda.stream(s):
        graphed.draw_grads(1)
        step_dev.fill_(1)
        graphed.handle.step(graphed.table(), **hp)          # t = 1 eagerly: the table's first use
        s.synchronize()
        with torch.cuda.graph(g, stream=s):
            step_dev.add_(1)
            graphed.handle.step(graphed.table(), **hp)
    for t in range(1, 8):
        eager.draw_grads(t)
        oj.step([H.to_np(x) for x in eager.grads], t)
        eager.step(t)
        if t > 1:
            with torch.cuda.stream(s):
                graphed.draw_grads(t)
                g.replay()
                s.synchronize()
        graphed.handle.device_status()
        assert int(step_dev.item()) == t
        H.compare_job(graphed, oj, REL_1STEP * t, f"graph t={t}")
        for x, y in zip(eager.states, graphed.states):
            assert torch.equal(x.m_codes, y.m_codes) and torch.equal(x.v_codes, y.v_codes)


@pytest.mark.parametrize("seed", range(24))
def test_random_tables_against_the_oracle(H, O, seed):
    """Randomised tables: sizes from 1 element to a few tiles, every block size, widths 2..32 on both
    sides of the step (so width changes, raw fp32 states and packed states mix in one call), all three
    gradient types, both variants of the v code, per-tensor weight decay, AdamW and L2 mode, with and
    without statistics.  Three steps each, codes and scales bit for bit."""
    import oracle
    rng = np.random.RandomState(1000 + seed)
    widths = [2, 3, 4, 8, 16, 32]
    for case in range(6):
        L = int(rng.randint(1, 7))
        block = int(rng.choice([128, 256, 512]))
        gdt = [torch.float32, torch.bfloat16, torch.float16][int(rng.randint(0, 3))]
        decoupled = bool(rng.randint(0, 2))
        sizes = [int(rng.choice([1, 7, 127, 128, 129, 1000, 4095, 4096, 4097, 4096 * 2 + 333, 4096 * 3])) if rng.rand() < 0.6
                 else int(rng.randint(1, 20000)) for _ in range(L)]
        vlog = [int(rng.randint(0, 2)) for _ in range(L)]
        wds = [float(rng.choice([0.0, 0.01, 0.1])) for _ in range(L)]
        bits = [(int(rng.choice(widths)), int(rng.choice(widths))) for _ in range(L)]
        gen = torch.Generator(device="cuda").manual_seed(int(rng.randint(0, 2 ** 31)))
        params = [torch.empty(n, device="cuda").normal_(0, 0.02, generator=gen) for n in sizes]
        states = [stq.alloc_state(n, block, bm, bv, "cuda", vl) for n, (bm, bv), vl in zip(sizes, bits, vlog)]
        h = stq.Handle()
        h.init_state(stq.table([stq.make_row(n, block, None, s) for n, s in zip(sizes, states)]))
        theta = [H.to_np(p) for p in params]
        ostates = [oracle.new_state(n, block, bm, bv) for n, (bm, bv) in zip(sizes, bits)]
        upd = [np.abs(t) for t in theta]
        # mixed-precision extras on some tables: a loss scale (not always a power of two) and a working copy
        amp = rng.rand() < 0.4
        S = float(rng.choice([1024.0, 3.0, 65536.0])) if amp else 1.0
        inv = torch.tensor([np.float32(1.0 / S)], dtype=torch.float32, device="cuda") if amp else None
        lp_dt = [None, torch.bfloat16, torch.float16][int(rng.randint(0, 3))] if amp else None
        lps = [torch.zeros(n, dtype=lp_dt, device="cuda") if lp_dt is not None else None for n in sizes]
        for t in (1, 2, 3):
            scale = 10.0 ** rng.uniform(-5, -2) * (S if gdt != torch.float16 else min(S, 1024.0))
            grads = [(torch.empty(n, device="cuda").normal_(0, 1.0, generator=gen) * scale).to(gdt) for n in sizes]
            new_bits = [(int(rng.choice(widths)), int(rng.choice(widths))) if rng.rand() < 0.3 else b for b in bits]
            out = [s if nb == b else stq.alloc_state(n, block, nb[0], nb[1], "cuda", vl)
                   for s, nb, b, n, vl in zip(states, new_bits, bits, sizes, vlog)]
            want_stats = bool(rng.randint(0, 2))
            rows = [stq.make_row(n, block, s, o, p, g, wd, lp)
                    for n, s, o, p, g, wd, lp in zip(sizes, states, out, params, grads, wds, lps)]
            h.step(stq.table(rows), lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, t=t, grad_dtype=stq.grad_dtype_of(grads[0]),
                   decoupled_wd=decoupled, flags=stq.WITH_STATS if want_stats else 0, inv_grad_scale=inv)
            got_stats = h.layer_stats(L) if want_stats else None
            h.device_status()
            states, bits = out, new_bits
            for i in range(L):
                before = theta[i].copy()
                ostates[i], st = oracle.step(theta[i], H.to_np(grads[i]), ostates[i], block, lr=1e-3, beta1=0.9, beta2=0.999,
                                             eps=1e-8, weight_decay=wds[i], t=t, bits_m_out=bits[i][0], bits_v_out=bits[i][1],
                                             decoupled_wd=decoupled, want_stats=want_stats, fp16_grad=(gdt == torch.float16),
                                             v_mode=oracle.LOG_PL if vlog[i] else oracle.LOG,
                                             inv_grad_scale=float(np.float32(1.0 / S)))
                upd[i] = np.maximum(upd[i], np.maximum(np.abs(theta[i]), np.abs(theta[i] - before)))
                tag = f"seed {seed} case {case} t={t} tensor {i} n={sizes[i]} B={block} bits {bits[i]} {gdt}"
                H.assert_states_equal(states[i], ostates[i], tag)
                H.assert_theta_close(params[i], theta[i], REL_1STEP * t, tag, upd=upd[i])
                if want_stats:
                    H.assert_stats_close(got_stats[i:i + 1], st[None, :], tag)
                if lps[i] is not None:
                    assert torch.equal(lps[i], params[i].to(lp_dt)), tag + " working copy"
                if not decoupled:
                    # L2 mode feeds the parameters back into the moments (g + lambda * theta), and the parameters
                    # agree to rounding, not to the bit: each step is checked from identical inputs
                    theta[i] = H.to_np(params[i])


@pytest.mark.parametrize("seed", range(6))
def test_random_repacks_and_statistics_against_the_oracle(H, O, seed):
    """Randomised width transitions without a step (stq_repack, including to and from raw fp32 states and
    in both variants of the v code) and the statistics-only pass, on states that two steps have filled."""
    import oracle
    rng = np.random.RandomState(2000 + seed)
    widths = [2, 3, 4, 8, 16, 32]
    for case in range(6):
        L = int(rng.randint(1, 6))
        block = int(rng.choice([128, 256, 512]))
        gdt = [torch.float32, torch.bfloat16, torch.float16][int(rng.randint(0, 3))]
        sizes = [int(rng.choice([1, 129, 4095, 4096, 4097, 4096 * 2 + 333])) if rng.rand() < 0.5 else int(rng.randint(1, 15000))
                 for _ in range(L)]
        vlog = [int(rng.randint(0, 2)) for _ in range(L)]
        bits = [(int(rng.choice(widths)), int(rng.choice(widths))) for _ in range(L)]
        gen = torch.Generator(device="cuda").manual_seed(int(rng.randint(0, 2 ** 31)))
        params = [torch.empty(n, device="cuda").normal_(0, 0.02, generator=gen) for n in sizes]
        states = [stq.alloc_state(n, block, bm, bv, "cuda", vl) for n, (bm, bv), vl in zip(sizes, bits, vlog)]
        h = stq.Handle()
        h.init_state(stq.table([stq.make_row(n, block, None, s) for n, s in zip(sizes, states)]))
        theta = [H.to_np(p) for p in params]
        ostates = [oracle.new_state(n, block, bm, bv) for n, (bm, bv) in zip(sizes, bits)]
        for t in (1, 2):
            grads = [(torch.empty(n, device="cuda").normal_(0, 1.0, generator=gen) * 10.0 ** rng.uniform(-4, -2)).to(gdt)
                     for n in sizes]
            rows = [stq.make_row(n, block, s, s, p, g, 0.01) for n, s, p, g in zip(sizes, states, params, grads)]
            h.step(stq.table(rows), lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, t=t, grad_dtype=stq.grad_dtype_of(grads[0]))
            for i in range(L):
                ostates[i], _ = oracle.step(theta[i], H.to_np(grads[i]), ostates[i], block, lr=1e-3, beta1=0.9, beta2=0.999,
                                            eps=1e-8, weight_decay=0.01, t=t, fp16_grad=(gdt == torch.float16),
                                            v_mode=oracle.LOG_PL if vlog[i] else oracle.LOG)
        # statistics alone, on the last gradients
        h.grad_stats(stq.table([stq.make_row(n, block, s, s, p, g) for n, s, p, g in zip(sizes, states, params, grads)]),
                     stq.grad_dtype_of(grads[0]))
        got = h.layer_stats(L)
        want = np.stack([oracle.grad_stats(H.to_np(g), fp16=(gdt == torch.float16)) for g in grads])
        H.assert_stats_close(got, want, f"seed {seed} case {case} statistics")
        # two repacks in a row
        for hop in range(2):
            new_bits = [(int(rng.choice(widths)), int(rng.choice(widths))) for _ in range(L)]
            out = [stq.alloc_state(n, block, nb[0], nb[1], "cuda", vl) for n, nb, vl in zip(sizes, new_bits, vlog)]
            h.repack(stq.table([stq.make_row(n, block, s, o) for n, s, o in zip(sizes, states, out)]))
            h.device_status()
            for i in range(L):
                st = ostates[i]
                n = sizes[i]
                vm = oracle.LOG_PL if vlog[i] else oracle.LOG
                mc, ms = oracle.repack(st.m_codes, st.m_scales, st.bits_m, new_bits[i][0], n, block, oracle.LINEAR)
                vc, vs = oracle.repack(st.v_codes, st.v_scales, st.bits_v, new_bits[i][1], n, block, vm)
                ostates[i] = oracle.State(mc, ms, new_bits[i][0], vc, vs, new_bits[i][1])
                H.assert_states_equal(out[i], ostates[i], f"seed {seed} case {case} hop {hop} tensor {i} n={n} B={block} "
                                                          f"{bits[i]} -> {new_bits[i]} pl={vlog[i]}")
            states, bits = out, new_bits


@pytest.mark.parametrize("seed", range(3))
def test_random_medium_tables_many_bodies_in_one_launch(H, O, seed):
    """Forty tensors of tens to hundreds of tiles with random widths, so that one launch runs many fused
    bodies, the runtime-width body (a third of the tensors change width every step) and the generic
    kernel side by side; five steps with statistics on every other one."""
    import oracle
    rng = np.random.RandomState(3000 + seed)
    widths = [2, 3, 4, 8, 16]
    L = 40
    block = [128, 256, 128][seed]
    gdt = [torch.bfloat16, torch.float32, torch.float16][seed]
    sizes = [int(rng.randint(20000, 200000)) for _ in range(L)]
    vlog = [int(rng.randint(0, 2)) for _ in range(L)]
    bits = [(int(rng.choice(widths)), int(rng.choice(widths))) for _ in range(L)]
    gen = torch.Generator(device="cuda").manual_seed(seed)
    params = [torch.empty(n, device="cuda").normal_(0, 0.02, generator=gen) for n in sizes]
    states = [stq.alloc_state(n, block, bm, bv, "cuda", vl) for n, (bm, bv), vl in zip(sizes, bits, vlog)]
    h = stq.Handle()
    h.init_state(stq.table([stq.make_row(n, block, None, s) for n, s in zip(sizes, states)]))
    theta = [H.to_np(p) for p in params]
    ostates = [oracle.new_state(n, block, bm, bv) for n, (bm, bv) in zip(sizes, bits)]
    upd = [np.abs(t) for t in theta]
    for t in range(1, 6):
        grads = [(torch.empty(n, device="cuda").normal_(0, 1.0, generator=gen) * 10.0 ** rng.uniform(-4, -2)).to(gdt) for n in sizes]
        new_bits = [(int(rng.choice(widths)), int(rng.choice(widths))) if rng.rand() < 0.33 else b for b in bits]
        out = [s if nb == b else stq.alloc_state(n, block, nb[0], nb[1], "cuda", vl)
               for s, nb, b, n, vl in zip(states, new_bits, bits, sizes, vlog)]
        want_stats = t % 2 == 0
        h.step(stq.table([stq.make_row(n, block, s, o, p, g, 0.01) for n, s, o, p, g in zip(sizes, states, out, params, grads)]),
               lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, t=t, grad_dtype=stq.grad_dtype_of(grads[0]),
               flags=stq.WITH_STATS if want_stats else 0)
        got = h.layer_stats(L) if want_stats else None
        h.device_status()
        states, bits = out, new_bits
        for i in range(L):
            before = theta[i].copy()
            ostates[i], st = oracle.step(theta[i], H.to_np(grads[i]), ostates[i], block, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8,
                                         weight_decay=0.01, t=t, bits_m_out=bits[i][0], bits_v_out=bits[i][1],
                                         want_stats=want_stats, fp16_grad=(gdt == torch.float16),
                                         v_mode=oracle.LOG_PL if vlog[i] else oracle.LOG)
            upd[i] = np.maximum(upd[i], np.maximum(np.abs(theta[i]), np.abs(theta[i] - before)))
            tag = f"seed {seed} t={t} tensor {i} n={sizes[i]} bits {bits[i]} pl={vlog[i]}"
            H.assert_states_equal(states[i], ostates[i], tag)
            H.assert_theta_close(params[i], theta[i], REL_1STEP * t, tag, upd=upd[i])
            if want_stats:
                H.assert_stats_close(got[i:i + 1], st[None, :], tag)


def test_pending_statistics_are_dropped_when_the_table_changes(H, O):
    """Sums taken with one table cannot be finished with another table's tile and segment maps: a call with
    a different table in between makes stq_layer_stats report the call order instead of wrong sums."""
    shapes = [("a", (4096 * 3 + 5,)), ("b", (4096,)), ("c", (900,))]
    w = W.Workload("order", tuple(shapes), 128, "fp32", "normal", scale_log10=(-3.0, -3.0), seed=5)
    job = Job(w, [4, 8, 4], [4, 4, 8])
    oj = H.OracleJob(job)
    job.draw_grads(1)
    st_o = oj.step([H.to_np(g) for g in job.grads], 1, want_stats=True)
    job.step(1, stats=True)
    job.step(2)                                   # the same table again: the sums of step 1 stay pending
    H.assert_stats_close(job.layer_stats(), st_o, "still pending after a plain step")
    job.step(3, stats=True)
    job.repack(([8, 8, 4], [4, 4, 8]))            # another table through the same handle
    with pytest.raises(stq.StqError) as err:
        job.layer_stats()
    assert err.value.code == stq.E_STATE
    job.draw_grads(4)
    job.step(4, stats=True)                       # and the next request works as usual
    want = np.stack([O.grad_stats(H.to_np(g)) for g in job.grads])
    H.assert_stats_close(job.layer_stats(), want, "after the drop")


@pytest.mark.parametrize("block", [32, 64, 512, 1024])
@pytest.mark.parametrize("bits", [(4, 4), (3, 8), (8, 2), (16, 3), (2, 16), (32, 4), (8, 32)])
def test_blocks_from_32_to_1024(H, O, block, bits):
    """The block sizes that the generic kernel serves: a row of 128 elements holds four or two blocks (32, 64),
    or a block spans a whole warp (512) or two neighbouring warps (1024), including ragged last blocks that
    end inside a lane group, a width change inside a step and a re-pack."""
    import oracle
    for n, gdt, v_log in ((4096 * 2 + 1024 + 333, "fp32", "poly"), (4096 + 37, "bf16", "pl"), (29, "bf16", "poly"),
                          (1024 * 3, "fp32", "poly")):
        if v_log == "pl" and 32 in bits:
            continue
        from dataclasses import replace
        w = replace(_single(n, block, gdt, seed=block + n), v_log=v_log)
        job = Job(w, [bits[0]], [bits[1]])
        oj = H.OracleJob(job)
        H.compare_job(job, oj, 0.0, f"B={block} n={n} init")
        for t in (1, 2, 3):
            job.draw_grads(t)
            new_bits = ([8], [4]) if t == 3 else None          # step 3 writes other widths
            st = oj.step([H.to_np(g) for g in job.grads], t, want_stats=True, new_bits=new_bits)
            job.step(t, stats=True, new_bits=new_bits)
            H.compare_job(job, oj, REL_1STEP * t, f"B={block} n={n} t={t}")
            H.assert_stats_close(job.layer_stats(), st, f"B={block} n={n}")
        job.repack(([bits[0]], [bits[1]]))
        oj.repack(([bits[0]], [bits[1]]))
        H.compare_job(job, oj, REL_1STEP * 3, f"B={block} n={n} repack")


def test_blocks_of_every_size_in_one_table(H, O):
    """One table whose tensors differ in block size cannot exist (the block is a property of the workload's
    table rows, and each row carries its own): mix them and check every row against the oracle."""
    import oracle
    dev = "cuda"
    sizes = [(4096 * 2 + 77, 32), (4096 + 512, 64), (4096 * 3, 128), (9000, 256), (4096 * 2 + 600, 512), (4096 * 2 + 1500, 1024)]
    h = stq.Handle()
    gen = torch.Generator(device=dev).manual_seed(11)
    params = [torch.randn(n, device=dev, generator=gen) * 0.02 for n, _ in sizes]
    states = [stq.alloc_state(n, b, 4, 8, dev) for n, b in sizes]
    h.init_state(stq.table([stq.make_row(n, b, None, s) for (n, b), s in zip(sizes, states)]))
    o_theta = [H.to_np(p) for p in params]
    o_states = [oracle.new_state(n, b, 4, 8) for n, b in sizes]
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8)
    for t in (1, 2, 3):
        grads = [torch.randn(n, device=dev, generator=gen) * 1e-3 for n, _ in sizes]
        h.step(stq.table([stq.make_row(n, b, s, s, p, g, 0.01) for (n, b), s, p, g in zip(sizes, states, params, grads)]),
               t=t, flags=stq.WITH_STATS, **hp)
        got = h.layer_stats(len(sizes))
        for i, (n, b) in enumerate(sizes):
            o_states[i], st = oracle.step(o_theta[i], H.to_np(grads[i]), o_states[i], b, weight_decay=0.01, t=t,
                                          want_stats=True, **hp)
            H.assert_states_equal(states[i], o_states[i], f"B={b} t={t}")
            H.assert_theta_close(params[i], o_theta[i], REL_1STEP * t, f"B={b} t={t}", upd=np.abs(o_theta[i]) + 1e-3)
            H.assert_stats_close(got[i:i + 1], st[None, :], f"B={b} t={t}")
    h.close()


# ---- the stochastic-rounding and the two-scale code of the second moment -------------------------------------
@pytest.mark.parametrize("v_log", ["sr", "ts"])
@pytest.mark.parametrize("bv", [2, 3, 4, 8, 16])
@pytest.mark.parametrize("bm,block,gdt", [(4, 128, "bf16"), (16, 256, "fp32"), (3, 64, "fp32"), (8, 1024, "bf16"), (32, 128, "fp32")])
def test_sr_and_ts_codes_every_width(H, O, v_log, bv, bm, block, gdt):
    """Both codes at every width of the second moment, with ragged sizes, fused statistics, a width change
    inside a step and a re-pack: codes and scales (two per block for "ts") bit for bit, the random words of
    "sr" included."""
    from dataclasses import replace
    for n in (4096 * 2 + 128 * 5 + 52, 999):
        w = replace(_single(n, block, gdt, seed=bm * 100 + bv), v_log=v_log)
        job = Job(w, [bm], [bv])
        oj = H.OracleJob(job)
        H.compare_job(job, oj, 0.0, "init")
        for t in (1, 2, 3, 4):
            job.draw_grads(t)
            new_bits = ([8], [4 if bv != 4 else 8]) if t == 3 else None
            st = oj.step([H.to_np(g) for g in job.grads], t, want_stats=True, new_bits=new_bits)
            job.step(t, stats=True, new_bits=new_bits)
            H.compare_job(job, oj, REL_1STEP * t, f"{v_log} n={n} t={t}")
            H.assert_stats_close(job.layer_stats(), st, v_log)
        job.repack(([bm], [bv]))
        oj.repack(([bm], [bv]))
        H.compare_job(job, oj, REL_1STEP * 4, f"{v_log} n={n} repack")


def test_all_four_codes_in_one_table_and_extreme_values(H, O):
    """Tensors coded with each of the four readings side by side in one call; zero blocks, denormal and huge
    gradients, one outlier per block."""
    import oracle
    dev, block, n = "cuda", 128, 4096 * 2 + 128 * 3 + 7
    modes = [("poly", oracle.LOG), ("pl", oracle.LOG_PL), ("sr", oracle.LOG_SR), ("ts", oracle.LOG_TS)] * 2
    widths = [(4, 8), (8, 16), (4, 4), (3, 8), (16, 2), (2, 8), (8, 16), (4, 2)]
    h = stq.Handle()
    gen = torch.Generator(device=dev).manual_seed(3)
    params = [torch.randn(n, device=dev, generator=gen) * 0.02 for _ in modes]
    states = [stq.alloc_state(n, block, bm, bv, dev, stq.VLOG_BY_NAME[name]) for (name, _), (bm, bv) in zip(modes, widths)]
    h.init_state(stq.table([stq.make_row(n, block, None, s) for s in states]))
    o_theta = [H.to_np(p) for p in params]
    o_states = [oracle.new_state(n, block, bm, bv, vm) for (_, vm), (bm, bv) in zip(modes, widths)]
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8)
    for t in (1, 2, 3):
        grads = []
        for i in range(len(modes)):
            x = torch.randn(n, generator=gen, device=dev) * 1e-3
            blk = x[:n // block * block].view(-1, block)
            blk[0::7] = 0.0
            blk[1::7] *= 1e-42
            blk[2::7] *= 1e-25
            blk[3::7] *= 1e15
            blk[4::7, 5] = 3e3
            blk[5::7, ::2] = 0.0                                   # zeros among ordinary values: the floor of "ts"
            grads.append(x)
        h.step(stq.table([stq.make_row(n, block, s, s, p, g, 0.01, sr_id=i)
                          for i, (s, p, g) in enumerate(zip(states, params, grads))]), t=t, sr_seed=77, **hp)
        for i, (_, vm) in enumerate(modes):
            o_states[i], _ = oracle.step(o_theta[i], H.to_np(grads[i]), o_states[i], block, weight_decay=0.01, t=t,
                                         v_mode=vm, sr_seed=77, tensor_index=i, **hp)
            H.assert_states_equal(states[i], o_states[i], f"{modes[i][0]} t={t}")
            H.assert_theta_close(params[i], o_theta[i], REL_1STEP * t, f"{modes[i][0]} t={t}", upd=np.abs(o_theta[i]) + 1.0)
    h.close()


def test_stochastic_rounding_seeds_and_call_rules(H, O):
    from dataclasses import replace
    w = replace(_single(4096 * 2 + 300, 128, "bf16", seed=4), v_log="sr")
    codes = []
    for seed in (1, 1, 2):
        job = Job(w, [4], [4])
        job.sr_seed = seed
        job.draw_grads(1)
        job.step(1)
        torch.cuda.synchronize()
        codes.append(job.states[0].v_codes.clone())
    assert torch.equal(codes[0], codes[1]) and not torch.equal(codes[0], codes[2])
    # the random words are keyed on the host's step count: a step count kept on the device is refused
    step_dev = torch.ones(1, dtype=torch.int64, device="cuda")
    with pytest.raises(stq.StqError) as err:
        job.handle.step(job.table(), **{**job.hp(2), "step_dev": step_dev})
    assert err.value.code == -9
    # sizes: the two-scale code keeps two floats per block
    assert stq.lib().stq_v_scales_bytes(1000, 128, stq.VLOG_TS) == 2 * stq.scales_bytes(1000, 128)
    assert stq.lib().stq_v_scales_bytes(1000, 128, stq.VLOG_SR) == stq.scales_bytes(1000, 128)


@pytest.mark.parametrize("seed", range(12))
def test_random_tables_with_every_code_and_block_size(H, O, seed):
    """Randomised tables in which every row draws its own block size (32..1024) and its own code of the second
    moment (default, "pl", "sr", "ts"), next to random sizes, widths 2..32 with width changes, gradient types,
    weight decay and statistics.  Three steps each, codes and scales (and random words) bit for bit."""
    import oracle
    rng = np.random.RandomState(5000 + seed)
    widths = [2, 3, 4, 8, 16, 32]
    modes = [oracle.LOG, oracle.LOG_PL, oracle.LOG_SR, oracle.LOG_TS]
    for case in range(5):
        L = int(rng.randint(1, 8))
        gdt = [torch.float32, torch.bfloat16, torch.float16][int(rng.randint(0, 3))]
        sizes = [int(rng.choice([1, 31, 33, 127, 129, 1000, 1024, 4095, 4096, 4097, 4096 * 2 + 333, 4096 * 4])) if rng.rand() < 0.6
                 else int(rng.randint(1, 30000)) for _ in range(L)]
        blocks = [int(rng.choice([32, 64, 128, 128, 256, 256, 512, 1024])) for _ in range(L)]
        vlog = [int(rng.randint(0, 4)) for _ in range(L)]
        wds = [float(rng.choice([0.0, 0.01, 0.1])) for _ in range(L)]
        bits = [(int(rng.choice(widths)), int(rng.choice(widths))) for _ in range(L)]
        sr_seed = int(rng.randint(0, 2 ** 31)) * 977 + 5
        gen = torch.Generator(device="cuda").manual_seed(int(rng.randint(0, 2 ** 31)))
        params = [torch.empty(n, device="cuda").normal_(0, 0.02, generator=gen) for n in sizes]
        states = [stq.alloc_state(n, b, bm, bv, "cuda", vl) for n, b, (bm, bv), vl in zip(sizes, blocks, bits, vlog)]
        h = stq.Handle()
        h.init_state(stq.table([stq.make_row(n, b, None, s) for n, b, s in zip(sizes, blocks, states)]))
        theta = [H.to_np(p) for p in params]
        ostates = [oracle.new_state(n, b, bm, bv, modes[vl]) for n, b, (bm, bv), vl in zip(sizes, blocks, bits, vlog)]
        upd = [np.abs(t) for t in theta]
        for t in (1, 2, 3):
            scale = 10.0 ** rng.uniform(-5, -2)
            grads = [(torch.empty(n, device="cuda").normal_(0, 1.0, generator=gen) * scale).to(gdt) for n in sizes]
            new_bits = [(int(rng.choice(widths)), int(rng.choice(widths))) if rng.rand() < 0.25 else b for b in bits]
            out = [s if nb == b else stq.alloc_state(n, blk, nb[0], nb[1], "cuda", vl)
                   for s, nb, b, n, blk, vl in zip(states, new_bits, bits, sizes, blocks, vlog)]
            want_stats = bool(rng.randint(0, 2))
            rows = [stq.make_row(n, blk, s, o, p, g, wd, sr_id=i + 3)
                    for i, (n, blk, s, o, p, g, wd) in enumerate(zip(sizes, blocks, states, out, params, grads, wds))]
            h.step(stq.table(rows), lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, t=t, grad_dtype=stq.grad_dtype_of(grads[0]),
                   flags=stq.WITH_STATS if want_stats else 0, sr_seed=sr_seed)
            got_stats = h.layer_stats(L) if want_stats else None
            h.device_status()
            states, bits = out, new_bits
            for i in range(L):
                before = theta[i].copy()
                ostates[i], st = oracle.step(theta[i], H.to_np(grads[i]), ostates[i], blocks[i], lr=1e-3, beta1=0.9,
                                             beta2=0.999, eps=1e-8, weight_decay=wds[i], t=t, bits_m_out=bits[i][0],
                                             bits_v_out=bits[i][1], want_stats=want_stats, fp16_grad=(gdt == torch.float16),
                                             v_mode=modes[vlog[i]], sr_seed=sr_seed, tensor_index=i + 3)
                upd[i] = np.maximum(upd[i], np.maximum(np.abs(theta[i]), np.abs(theta[i] - before)))
                tag = (f"seed {seed} case {case} t={t} tensor {i} n={sizes[i]} B={blocks[i]} bits {bits[i]} "
                       f"code {vlog[i]} {gdt}")
                H.assert_states_equal(states[i], ostates[i], tag)
                H.assert_theta_close(params[i], theta[i], REL_1STEP * t, tag, upd=upd[i])
                if want_stats:
                    H.assert_stats_close(got_stats[i:i + 1], st[None, :], tag)
        h.close()


@pytest.mark.parametrize("seed", range(4))
def test_random_medium_tables_every_code_in_one_launch(H, O, seed):
    """Thirty-six tensors of tens to hundreds of tiles, each with its own code of the second moment (default,
    "pl", "sr", "ts"), its own block size (mostly 128 and 256, some 64 and 512) and random widths, a quarter of
    them changing width every step: one step runs the three work lists of the main kernel and the generic
    kernel side by side.  Some tables carry the mixed-precision extras (loss scale, working copy).  Four
    steps, statistics on every other one; codes, scales and random words bit for bit."""
    import oracle
    rng = np.random.RandomState(7000 + seed)
    widths = [2, 3, 4, 8, 16]
    modes = [oracle.LOG, oracle.LOG_PL, oracle.LOG_SR, oracle.LOG_TS]
    L = 36
    gdt = [torch.bfloat16, torch.float32, torch.float16][seed % 3]
    sizes = [int(rng.randint(20000, 160000)) for _ in range(L)]
    blocks = [int(rng.choice([128, 128, 128, 256, 256, 256, 64, 512])) for _ in range(L)]
    vlog = [int(rng.randint(0, 4)) for _ in range(L)]
    bits = [(int(rng.choice(widths)), int(rng.choice(widths))) for _ in range(L)]
    sr_seed = int(rng.randint(0, 2 ** 31)) * 1013 + 7
    gen = torch.Generator(device="cuda").manual_seed(100 + seed)
    params = [torch.empty(n, device="cuda").normal_(0, 0.02, generator=gen) for n in sizes]
    states = [stq.alloc_state(n, b, bm, bv, "cuda", vl) for n, b, (bm, bv), vl in zip(sizes, blocks, bits, vlog)]
    h = stq.Handle()
    h.init_state(stq.table([stq.make_row(n, b, None, s) for n, b, s in zip(sizes, blocks, states)]))
    theta = [H.to_np(p) for p in params]
    ostates = [oracle.new_state(n, b, bm, bv, modes[vl]) for n, b, (bm, bv), vl in zip(sizes, blocks, bits, vlog)]
    upd = [np.abs(t) for t in theta]
    amp = seed % 2 == 1
    S = 1024.0 if amp else 1.0
    inv = torch.tensor([np.float32(1.0 / S)], dtype=torch.float32, device="cuda") if amp else None
    lp_dt = torch.bfloat16 if amp else None
    lps = [torch.zeros(n, dtype=lp_dt, device="cuda") if amp else None for n in sizes]
    for t in range(1, 5):
        scale = 10.0 ** rng.uniform(-4, -2) * S
        grads = [(torch.empty(n, device="cuda").normal_(0, 1.0, generator=gen) * scale).to(gdt) for n in sizes]
        new_bits = [(int(rng.choice(widths)), int(rng.choice(widths))) if rng.rand() < 0.25 else b for b in bits]
        out = [s if nb == b else stq.alloc_state(n, blk, nb[0], nb[1], "cuda", vl)
               for s, nb, b, n, blk, vl in zip(states, new_bits, bits, sizes, blocks, vlog)]
        want_stats = t % 2 == 0
        rows = [stq.make_row(n, blk, s, o, p, g, 0.01, lp, sr_id=i)
                for i, (n, blk, s, o, p, g, lp) in enumerate(zip(sizes, blocks, states, out, params, grads, lps))]
        h.step(stq.table(rows), lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, t=t, grad_dtype=stq.grad_dtype_of(grads[0]),
               flags=stq.WITH_STATS if want_stats else 0, sr_seed=sr_seed, inv_grad_scale=inv)
        got = h.layer_stats(L) if want_stats else None
        h.device_status()
        states, bits = out, new_bits
        for i in range(L):
            before = theta[i].copy()
            ostates[i], st = oracle.step(theta[i], H.to_np(grads[i]), ostates[i], blocks[i], lr=1e-3, beta1=0.9, beta2=0.999,
                                         eps=1e-8, weight_decay=0.01, t=t, bits_m_out=bits[i][0], bits_v_out=bits[i][1],
                                         want_stats=want_stats, fp16_grad=(gdt == torch.float16), v_mode=modes[vlog[i]],
                                         sr_seed=sr_seed, tensor_index=i, inv_grad_scale=float(np.float32(1.0 / S)))
            upd[i] = np.maximum(upd[i], np.maximum(np.abs(theta[i]), np.abs(theta[i] - before)))
            tag = f"seed {seed} t={t} tensor {i} n={sizes[i]} B={blocks[i]} bits {bits[i]} code {vlog[i]} {gdt}"
            H.assert_states_equal(states[i], ostates[i], tag)
            H.assert_theta_close(params[i], theta[i], REL_1STEP * t, tag, upd=upd[i])
            if want_stats:
                H.assert_stats_close(got[i:i + 1], st[None, :], tag)
            if amp:
                assert torch.equal(lps[i], params[i].to(lp_dt)), tag + " working copy"
    h.close()


@pytest.mark.parametrize("v_log", ["poly", "pl", "sr"])
@pytest.mark.parametrize("recipe", ["cfg3", "cfg5"])
def test_tile_padded_storage_gives_the_unpadded_results(H, O, recipe, v_log):
    """Storage padded with zeros to whole 4096-element tiles, padded lengths given to the library: the real
    elements' codes, scales (first blocks) and parameters are those of the oracle's run on the unpadded tensors,
    the gradient sums are unchanged, and a plain step is a single launch.  Small models with ragged tensor
    lengths (odd sizes, lengths below one block), width changes by stq_repack and inside the step (the ViT
    recipe), stochastic rounding keyed by the element's index in its tensor."""
    from dataclasses import replace
    from paper_2604_06836_b200.runner import Job
    shapes = W.small_vit() if recipe == "cfg3" else W.small_gpt2(d=100, n_layer=4, vocab=523)
    w = replace(W.scaled(W.config(recipe), shapes, steps=24), v_log=v_log)
    bm, bv, _ = W.draw_bits(w)
    job = Job(w, bm, bv, tile_padded=True)
    fo = H.FullOracle(job, range_elems=1 << 14, threads=4)
    fo.compare(0.0, "init")
    decisions = 0
    for t in range(1, 25):
        job.draw_grads(t)
        dec = t % 6 == 0
        new_bits = None
        if dec and w.churn > 0:
            nbm, nbv, _ = W.churn_bits(w, job.bits_m, job.bits_v, decisions)
            decisions += 1
            if decisions % 2 == 0:
                new_bits = (nbm, nbv)                    # inside the step
            else:
                job.repack((nbm, nbv))                   # between steps
                fo.repack((nbm, nbv))
        st_o = fo.step(t, new_bits=new_bits, want_stats=dec)
        n0 = job.handle.launch_count
        job.step(t, stats=dec, new_bits=new_bits)
        if not dec:
            assert job.handle.launch_count - n0 == 1
        fo.compare(REL_1STEP * t if t <= 10 else 1e-4, f"{recipe} {v_log} tile-padded t={t}")
        if dec:
            H.assert_stats_close(job.layer_stats(), st_o, f"{recipe} {v_log} t={t}")
    # the two-scale code keeps a block minimum, which padding inside a block would change: refused
    if any(n % w.block for n in w.numels):
        with pytest.raises(ValueError):
            Job(replace(w, v_log="ts"), bm, bv, tile_padded=True)

"""STQAdamW, the torch.optim wrapper that runs Algorithm 1 end to end (statistics, decision, update at the
new widths) on the library."""
import copy

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2604_06836_b200.optim import STQAdamW   # noqa: E402


def _mlp(seed=0, d=96):
    torch.manual_seed(seed)
    return torch.nn.Sequential(torch.nn.Linear(d, 4 * d), torch.nn.GELU(), torch.nn.Linear(4 * d, d),
                               torch.nn.LayerNorm(d), torch.nn.Linear(d, 8)).cuda()


def _batch(step, d=96):
    g = torch.Generator(device="cuda").manual_seed(100 + step)
    x = torch.randn(64, d, device="cuda", generator=g)
    y = torch.tanh(x[:, :8] * 2.0 - x[:, 8:16])
    return x, y


def test_raw_fp32_states_follow_library_adamw():
    """At 32-bit states the wrapper is AdamW: same parameters as torch.optim.AdamW on a real model."""
    a, b = _mlp(1), _mlp(1)
    oa = STQAdamW(a.parameters(), lr=2e-3, weight_decay=0.05, policy="fixed", init_bits=32)
    ob = torch.optim.AdamW(b.parameters(), lr=2e-3, weight_decay=0.05)
    for step in range(20):
        x, y = _batch(step)
        for m, o in ((a, oa), (b, ob)):
            o.zero_grad()
            torch.nn.functional.mse_loss(m(x), y).backward()
            o.step()
    for pa, pb in zip(a.parameters(), b.parameters()):
        scale = max(float(pb.detach().abs().max()), 1e-3)
        assert float((pa - pb).detach().abs().max()) <= 2e-5 * scale


def test_paper_policy_trains_and_resumes_bit_for_bit():
    model = _mlp(2)
    opt = STQAdamW(model.parameters(), lr=2e-3, weight_decay=0.01, policy="paper", interval=5, tau=20.0)
    assert opt.mean_bits() == 16.0
    losses, snap = [], None
    for step in range(40):
        if step == 17:
            snap = (copy.deepcopy(model.state_dict()), opt.state_dict())
        x, y = _batch(step)
        opt.zero_grad()
        loss = torch.nn.functional.mse_loss(model(x), y)
        loss.backward()
        opt.step()
        losses.append(float(loss.detach()))
    assert np.mean(losses[-5:]) < 0.7 * np.mean(losses[:5])
    assert set(opt.bits_m.tolist()) <= {4, 8, 16, 32} and (opt.bits_m == opt.bits_v).all()
    assert opt.last_scores is not None and opt.state_bytes() > 0
    # resume from the snapshot: the continuation reproduces the parameters exactly
    model2 = _mlp(3)
    model2.load_state_dict(snap[0])
    opt2 = STQAdamW(model2.parameters(), lr=2e-3, weight_decay=0.01, policy="paper", interval=5, tau=20.0)
    opt2.load_state_dict(snap[1])
    for step in range(17, 40):
        x, y = _batch(step)
        opt2.zero_grad()
        torch.nn.functional.mse_loss(model2(x), y).backward()
        opt2.step()
    for p, q in zip(model.parameters(), model2.parameters()):
        assert torch.equal(p, q)
    assert (opt.bits_m == opt2.bits_m).all()


@pytest.mark.parametrize("v_log", ["poly", "pl"])
def test_wrapper_matches_the_oracle_run_of_algorithm_1(v_log):
    """Same gradients into the wrapper and into the oracle's Algorithm 1 (statistics -> decision -> step at
    the new widths): codes and scales bit for bit, parameters to 1e-6 per step."""
    import harness as H
    import oracle
    torch.manual_seed(5)
    sizes = [4096 * 2 + 300, 777, 4096, 128 * 40]
    params = [torch.nn.Parameter(torch.randn(n, device="cuda") * 0.02) for n in sizes]
    wds = [0.01, 0.0]
    opt = STQAdamW([dict(params=params[:2], weight_decay=wds[0]), dict(params=params[2:], weight_decay=wds[1])],
                   lr=1e-3, policy="paper", interval=4, tau=8.0, v_log=v_log)
    vm = oracle.LOG_PL if v_log == "pl" else oracle.LOG
    theta = [H.to_np(p.data) for p in params]
    states = [oracle.new_state(n, 128, 16, 16) for n in sizes]
    pol = oracle.new_policy(0.1, 8.0, 1e-8)
    upd = [np.abs(t) for t in theta]
    scales = [1e-3, 3e-5, 1e-2, 2e-4]
    for t in range(1, 15):
        g = torch.Generator(device="cuda").manual_seed(t)
        for p, s in zip(params, scales):
            p.grad = torch.randn(p.numel(), device="cuda", generator=g) * s * (1.0 + 3.0 * (t % 3))
        grads = [H.to_np(p.grad) for p in params]
        bits = None
        if oracle.is_decision_step(t, 4):
            st = np.stack([oracle.grad_stats(x) for x in grads])
            bits, _ = oracle.decide(pol, st, t)
        opt.step()
        for i in range(len(sizes)):
            before = theta[i].copy()
            b = None if bits is None else int(bits[i])
            states[i], _ = oracle.step(theta[i], grads[i], states[i], 128, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8,
                                       weight_decay=wds[i // 2], t=t, bits_m_out=b, bits_v_out=b, v_mode=vm)
            upd[i] = np.maximum(upd[i], np.maximum(np.abs(theta[i]), np.abs(theta[i] - before)))
            H.assert_states_equal(opt.states[i], states[i], f"t={t} tensor {i}")
            H.assert_theta_close(params[i].data, theta[i], 1e-6 * t, f"t={t} tensor {i}", upd=upd[i])
        if bits is not None:
            assert (opt.bits_m == bits).all()


def test_fused_order_decides_on_the_previous_steps_gradients():
    """order="fused": the statistics of a decision step ride on the update before it, so the decision at
    step t sees the gradients of step t - 1 (t = 1 has none and takes a pre-pass).  Against the oracle."""
    import harness as H
    import oracle
    torch.manual_seed(6)
    sizes = [4096 * 2 + 300, 777, 4096]
    params = [torch.nn.Parameter(torch.randn(n, device="cuda") * 0.02) for n in sizes]
    opt = STQAdamW(params, lr=1e-3, weight_decay=0.01, policy="paper", interval=4, tau=8.0, order="fused")
    theta = [H.to_np(p.data) for p in params]
    states = [oracle.new_state(n, 128, 16, 16) for n in sizes]
    pol = oracle.new_policy(0.1, 8.0, 1e-8)
    upd = [np.abs(t) for t in theta]
    prev = None
    for t in range(1, 14):
        g = torch.Generator(device="cuda").manual_seed(50 + t)
        for k, p in enumerate(params):
            p.grad = torch.randn(p.numel(), device="cuda", generator=g) * (1e-3 * 10.0 ** (-k)) * (1.0 + 2.0 * (t % 4))
        grads = [H.to_np(p.grad) for p in params]
        bits = None
        if oracle.is_decision_step(t, 4):
            src = grads if t == 1 else prev
            st = np.stack([oracle.grad_stats(x) for x in src])
            bits, _ = oracle.decide(pol, st, t)
        opt.step()
        for i in range(len(sizes)):
            before = theta[i].copy()
            b = None if bits is None else int(bits[i])
            states[i], _ = oracle.step(theta[i], grads[i], states[i], 128, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8,
                                       weight_decay=0.01, t=t, bits_m_out=b, bits_v_out=b)
            upd[i] = np.maximum(upd[i], np.maximum(np.abs(theta[i]), np.abs(theta[i] - before)))
            H.assert_states_equal(opt.states[i], states[i], f"fused t={t} tensor {i}")
            H.assert_theta_close(params[i].data, theta[i], 1e-6 * t, f"fused t={t} tensor {i}", upd=upd[i])
        prev = grads


@pytest.mark.parametrize("order", ["paper", "fused"])
def test_a_skipped_step_leaves_no_trace(order):
    """Loss-scaled training: a step whose gradients overflowed is left out.  The step count, the bias
    corrections, the decision schedule and the running averages of the policy then follow the steps actually
    taken, so a run with overflow steps sprinkled in ends exactly where the run without them ends."""
    def run(skip_at):
        model = _mlp(5)
        opt = STQAdamW(model.parameters(), lr=2e-3, weight_decay=0.01, policy="paper", interval=4, tau=20.0,
                       order=order)
        opt.found_inf = torch.zeros(1, dtype=torch.float32, device="cuda")
        real = 0
        for it in range(14 + len(skip_at)):
            x, y = _batch(real)
            opt.zero_grad()
            torch.nn.functional.mse_loss(model(x), y).backward()
            if it in skip_at:
                for p in model.parameters():          # what an overflow leaves behind
                    p.grad.fill_(float("inf"))
                opt.found_inf.fill_(1.0)
            else:
                opt.found_inf.fill_(0.0)
                real += 1
            opt.step()
        return model, opt

    (ma, oa), (mb, ob) = run(()), run((2, 3, 7, 11))      # 3 and 7 sit right before decision steps (t = 4, 8)
    assert oa.t == ob.t == 14 and ob.skipped_steps == 4 and oa.skipped_steps == 0
    assert (oa.bits_m == ob.bits_m).all() and np.array_equal(oa.policy.state, ob.policy.state)
    assert np.isfinite(ob.policy.state).all()
    for pa, pb in zip(ma.parameters(), mb.parameters()):
        assert torch.equal(pa, pb)
    for sa, sb in zip(oa.states, ob.states):
        assert torch.equal(sa.m_codes, sb.m_codes) and torch.equal(sa.v_codes, sb.v_codes)
        assert torch.equal(sa.m_scales, sb.m_scales) and torch.equal(sa.v_scales, sb.v_scales)

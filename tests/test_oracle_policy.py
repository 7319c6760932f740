"""Pins for the oracle's gradient statistics and transition decision (Sec. 3.3-3.4, Algorithm 1)."""
import math
import os

import numpy as np

GOLD = os.path.join(os.path.dirname(__file__), "golden", "policy_pins.txt")


def pins():
    out = {}
    with open(GOLD) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                out[line[0]] = [float(v) for v in line[1:]]
    return out


def factors(stats):
    """(n, r, v) of Eq. 2, 3, 8 from the four sums, written out independently of the oracle."""
    sg, sa, sq, N = stats
    mu = sa / N
    var = max(sq / N - mu * mu, 0.0)
    return math.sqrt(sq / N), math.sqrt(var) / (mu + 1e-8), sq / N


def test_stats_closed_forms(O):
    c = 3e-3
    s = O.grad_stats(np.full(1000, c, np.float32))
    n, r, v = factors(s)
    cf = float(np.float32(c))
    assert abs(n - cf) < 1e-12 and r < 1e-6 and abs(v - cf * cf) < 1e-15 and s[3] == 1000
    assert abs(s[0] - 1000 * cf) < 1e-12
    g = np.full(1000, c, np.float32)
    g[::2] *= -1
    s = O.grad_stats(g)
    n, r, v = factors(s)
    assert abs(s[0]) < 1e-15 and abs(n - cf) < 1e-12 and r < 1e-6          # +-c: |g| constant
    a, b = 1.0, 3.0
    g = np.array([a, -b] * 500, np.float32)
    n, r, v = factors(O.grad_stats(g))
    assert abs(r - abs(a - b) / (a + b)) < 1e-7                             # two-valued |g|
    assert abs(v - (a * a + b * b) / 2) < 1e-12 and abs(n * n - v) < 1e-12
    g = np.random.default_rng(0).normal(0, 1e-3, 2_000_000).astype(np.float32)
    n, r, v = factors(O.grad_stats(g))
    assert abs(r - math.sqrt(math.pi / 2 - 1)) < 3e-3                       # half-normal CV
    assert abs(n - 1e-3) < 5e-6


def test_stats_bf16_input(O):
    import torch
    g = torch.randn(5000, generator=torch.Generator().manual_seed(0)) * 1e-3
    gb = g.to(torch.bfloat16)
    s = O.grad_stats(gb.view(torch.int16).numpy().view(np.uint16).copy())
    w = gb.to(torch.float64)
    np.testing.assert_allclose(s, [w.sum(), w.abs().sum(), (w * w).sum(), 5000], rtol=1e-12)


def _stats_for(n_l, r_l, N=1000):
    """Sums of a two-valued |g| vector with the requested RMS n and CV r (sum g = 0)."""
    # |g| in {mu(1+r), mu(1-r)} half/half: mean mu, std mu*r, mean square mu^2(1+r^2)
    mu = n_l / math.sqrt(1 + r_l * r_l)
    return [0.0, mu * N, n_l * n_l * N, float(N)]


def test_schedule(O):
    p = pins()
    early = int(p["early_steps"][0])
    for U in (5, 10, 20):
        for t in range(1, 60):
            assert O.is_decision_step(t, U) == (t % U == 0 or t < early)


def test_score_anchor_and_thresholds(O):
    p = pins()
    phi = p["phi"][0]
    th = p["thresholds"]
    L = 8
    stats = np.array([_stats_for(1e-3, 0.5)] * L)
    # alpha = 1 makes the running averages equal to this step's layer means: all ratios are 1
    pol = O.new_policy(alpha=1.0, tau=1e-9, eps_stat=0.0)
    bits, score = O.decide(pol, stats, t=1000)
    assert np.allclose(score, phi, atol=1e-9) and (bits == 8).all()
    # annealing factor: S(0) = 2 adds one bit of score; S(tau) = 1 + sech(1)
    pol = O.new_policy(alpha=1.0, tau=50.0, eps_stat=0.0)
    _, score = O.decide(pol, stats, t=0)
    assert np.allclose(score, phi + math.log2(p["S0"][0]), atol=1e-9)
    pol = O.new_policy(alpha=1.0, tau=50.0, eps_stat=0.0)
    _, score = O.decide(pol, stats, t=50)
    assert np.allclose(score, phi + math.log2(p["S_at_tau"][0]), atol=1e-9)
    # one layer k times "more intense" than the others: n ratio k/mean, v ratio k^2/mean
    for L, k, want in [(8, 1.0, 8), (8, 0.5, 4), (8, 8.0, 16), (4096, 1e6, 32)]:
        rows = [_stats_for(1e-3, 0.5)] * (L - 1) + [_stats_for(1e-3 * k, 0.5)]
        pol = O.new_policy(alpha=1.0, tau=1e-9, eps_stat=0.0)
        bits, score = O.decide(pol, np.array(rows), t=1000)
        nbar = (L - 1 + k) / L
        vbar = (L - 1 + k * k) / L
        expect = phi + math.log2(k / nbar) + math.log2(k * k / vbar)
        assert abs(score[-1] - expect) < 1e-9
        assert bits[-1] == want
        assert bits[-1] == (4 if expect < th[0] else 8 if expect < th[1] else 16 if expect < th[2] else 32)


def test_threshold_edges_are_lower_inclusive(O):
    # drive the score through the variation factor only: score = 7.2 + log2(r / rbar)
    for target, want in [(6.79, 4), (6.8, 8), (11.99, 8), (12.0, 16), (23.99, 16), (24.0, 32)]:
        # running averages are seeded by hand so a single layer can sit anywhere
        pol = O.new_policy(alpha=0.0, tau=1e-9, eps_stat=0.0)
        pol.n_ema, pol.v_ema = 1e-3, 1e-6
        r = 1e-4
        pol.r_ema = r / 2.0 ** (target - 7.2)
        bits, score = O.decide(pol, np.array([_stats_for(1e-3, r)]), t=10 ** 6)
        assert abs(score[0] - target) < 1e-6
        if abs(score[0] - target) < 1e-12 or target not in (6.8, 12.0, 24.0):
            assert bits[0] == want
        assert bits[0] == (4 if score[0] < 6.8 else 8 if score[0] < 12 else 16 if score[0] < 24 else 32)


def test_first_decision_with_zero_averages_and_dead_layer(O):
    alpha = 0.1
    L = 4
    rows = [_stats_for(1e-3, 0.5)] * (L - 1) + [[0.0, 0.0, 0.0, 1000.0]]   # last layer: zero gradient
    pol = O.new_policy(alpha=alpha, tau=1e-9, eps_stat=1e-8)
    bits, score = O.decide(pol, np.array(rows), t=1000)
    assert score[-1] == -math.inf and bits[-1] == 4 and not np.isnan(score).any()
    # averages started at 0, so they are alpha * (mean over layers)
    assert abs(pol.n_ema - alpha * 1e-3 * (L - 1) / L) < 1e-15
    assert abs(pol.v_ema - alpha * 1e-6 * (L - 1) / L) < 1e-18
    # second call keeps averaging
    n1 = pol.n_ema
    O.decide(pol, np.array(rows), t=1001)
    assert abs(pol.n_ema - (alpha * 1e-3 * (L - 1) / L + (1 - alpha) * n1)) < 1e-15


def test_cv_variants(O):
    # Eq. 3 uses the deviation of |g|; Algorithm 1 prints the deviation of g itself
    g = np.array([1.0, -1.0] * 500, np.float32)
    s = O.grad_stats(g)
    pol_a = O.new_policy(alpha=1.0, tau=1e-9, eps_stat=0.0, cv_of_signed=False)
    pol_b = O.new_policy(alpha=1.0, tau=1e-9, eps_stat=0.0, cv_of_signed=True)
    O.decide(pol_a, s[None, :], t=100)
    O.decide(pol_b, s[None, :], t=100)
    assert pol_a.r_ema == 0.0          # |g| is constant
    assert abs(pol_b.r_ema - 1.0) < 1e-12   # sigma(g) = 1, E|g| = 1

"""Pins for the oracle's AdamW step (Algorithm 1 inner loop) against library / textbook AdamW."""
import numpy as np
import pytest
import torch

HP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)


def textbook_adamw(theta, grads, *, lr, beta1, beta2, eps, weight_decay, decoupled=True):
    """Float64 AdamW exactly as printed in Algorithm 1 with unquantized states."""
    th = theta.astype(np.float64).copy()
    m = np.zeros_like(th)
    v = np.zeros_like(th)
    b1, b2 = beta1, beta2
    for t, g in enumerate(grads, start=1):
        g = g.astype(np.float64)
        if not decoupled:
            g = g + weight_decay * th
        m = b1 * m + (1 - b1) * g
        v = b2 * v + (1 - b2) * g * g
        mh = m / (1 - b1 ** t)
        vh = v / (1 - b2 ** t)
        decay = (1 - lr * weight_decay) if decoupled else 1.0
        th = th * decay - lr * mh / (np.sqrt(vh) + eps)
    return th, m, v


def test_32bit_state_matches_torch_adamw(O):
    """With raw fp32 states the oracle is plain AdamW: compare with torch.optim.AdamW."""
    rng = np.random.default_rng(0)
    n = 1000
    theta0 = rng.normal(0, 0.02, n).astype(np.float32)
    grads = [rng.normal(0, 1e-3, n).astype(np.float32) for _ in range(20)]
    p = torch.nn.Parameter(torch.from_numpy(theta0.copy()))
    opt = torch.optim.AdamW([p], lr=HP["lr"], betas=(HP["beta1"], HP["beta2"]), eps=HP["eps"],
                            weight_decay=HP["weight_decay"], foreach=False, fused=False)
    th = theta0.copy()
    st = O.new_state(n, 128, 32, 32)
    for t, g in enumerate(grads, start=1):
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        st, _ = O.step(th, g, st, 128, t=t, **HP)
    ref = p.detach().numpy()
    assert np.abs(th - ref).max() <= 2e-6 * np.abs(ref).max()
    s = opt.state[p]
    # torch forms m by lerp, so small elements differ by rounding relative to the tensor's scale
    em, ev = s["exp_avg"].numpy(), s["exp_avg_sq"].numpy()
    assert np.abs(st.m_codes.view(np.float32)[:n] - em).max() <= 1e-6 * np.abs(em).max()
    assert np.abs(st.v_codes.view(np.float32)[:n] - ev).max() <= 1e-6 * np.abs(ev).max()


def test_32bit_state_l2_mode_matches_torch_adam(O):
    rng = np.random.default_rng(1)
    n = 777
    theta0 = rng.normal(0, 0.02, n).astype(np.float32)
    grads = [rng.normal(0, 1e-3, n).astype(np.float32) for _ in range(10)]
    p = torch.nn.Parameter(torch.from_numpy(theta0.copy()))
    opt = torch.optim.Adam([p], lr=HP["lr"], betas=(HP["beta1"], HP["beta2"]), eps=HP["eps"],
                           weight_decay=HP["weight_decay"], foreach=False, fused=False)
    th = theta0.copy()
    st = O.new_state(n, 128, 32, 32)
    for t, g in enumerate(grads, start=1):
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        st, _ = O.step(th, g, st, 128, t=t, decoupled_wd=False, **HP)
    ref = p.detach().numpy()
    assert np.abs(th - ref).max() <= 2e-6 * np.abs(ref).max()


def _fma32(a, b, c):
    """Correctly rounded fp32 fma of python floats holding fp32 values, by exact rational arithmetic."""
    from fractions import Fraction
    x = Fraction(a) * Fraction(b) + Fraction(c)
    if x == 0:
        return np.float32(0.0)
    sign = -1 if x < 0 else 1
    x = abs(x)
    e = x.numerator.bit_length() - x.denominator.bit_length()      # 2^(e-1) < x < 2^(e+1)
    if Fraction(2) ** e > x:
        e -= 1
    e = max(e, -126)                                               # subnormal results share the smallest exponent
    scaled = x / Fraction(2) ** (e - 23)                           # significand with 24 bits before the point
    q, r = divmod(scaled.numerator, scaled.denominator)
    twice = 2 * r
    if twice > scaled.denominator or (twice == scaled.denominator and q % 2 == 1):
        q += 1
    return np.float32(sign * float(Fraction(q) * Fraction(2) ** (e - 23)))


def test_32bit_moments_are_the_fp32_recursion_bit_for_bit(O):
    """m_t = fma(b1, m, fl(c1*g)), v_t = fma(b2, v, fl(fl(c2*g)*g)) in fp32, with b = fp32(beta) and
    c = fp32(1 - beta) (the subtraction taken in double)."""
    rng = np.random.default_rng(2)
    n = 200
    th = rng.normal(0, 0.02, n).astype(np.float32)
    st = O.new_state(n, 128, 32, 32)
    m = np.zeros(n, np.float32)
    v = np.zeros(n, np.float32)
    b1, b2 = np.float32(0.9), np.float32(0.999)
    c1, c2 = np.float32(1 - 0.9), np.float32(1 - 0.999)
    for t in range(1, 5):
        g = rng.normal(0, 1e-3, n).astype(np.float32)
        st, _ = O.step(th, g, st, 128, t=t, **HP)
        new_m = c1 * g
        new_v = (c2 * g) * g
        assert new_m.dtype == np.float32 and new_v.dtype == np.float32
        m = np.array([_fma32(float(b1), float(a), float(c)) for a, c in zip(m, new_m)], np.float32)
        v = np.array([_fma32(float(b2), float(a), float(c)) for a, c in zip(v, new_v)], np.float32)
        assert (st.m_codes.view(np.float32)[:n] == m).all()
        assert (st.v_codes.view(np.float32)[:n] == v).all()


def test_16bit_states_track_textbook_adamw(O):
    """Brute force on tiny tensors: 16-bit block-quantized states stay close to textbook AdamW."""
    rng = np.random.default_rng(3)
    n = 512
    theta0 = rng.normal(0, 0.02, n).astype(np.float32)
    sigma = 1e-3
    grads = [(rng.choice([-1.0, 1.0], n) * sigma * rng.uniform(0.05, 1.0, n)).astype(np.float32)
             for _ in range(10)]
    th = theta0.copy()
    st = O.new_state(n, 128, 16, 16)
    for t, g in enumerate(grads, start=1):
        st, _ = O.step(th, g, st, 128, t=t, **HP)
        ref, _, _ = textbook_adamw(theta0, grads[:t], **HP)
        lim = 1e-3 if t == 1 else 5e-3
        assert np.abs(th - ref).max() <= lim * HP["lr"], (t, np.abs(th - ref).max() / HP["lr"])


@pytest.mark.parametrize("bits_m,bits_v", [(8, 4), (4, 3), (2, 2), (16, 8)])
def test_update_consumes_the_quantized_states(O, bits_m, bits_v):
    """theta_t is computed from the decoded new codes, not from the unquantized moments."""
    rng = np.random.default_rng(4)
    n = 128 * 5 + 40
    theta0 = rng.normal(0, 0.02, n).astype(np.float32)
    th = theta0.copy()
    st = O.new_state(n, 128, bits_m, bits_v)
    for t in range(1, 4):
        g = (rng.standard_t(4, n) * 1e-3).astype(np.float32)
        before = th.copy()
        st, _ = O.step(th, g, st, 128, t=t, **HP)
        mh = O.dequantize(st.m_codes, st.m_scales, n, bits_m, 128, O.LINEAR).astype(np.float64)
        vh = O.dequantize(st.v_codes, st.v_scales, n, bits_v, 128, O.LOG).astype(np.float64)
        b1, b2 = HP["beta1"], HP["beta2"]
        lr, wd, eps = (HP[k] for k in ("lr", "weight_decay", "eps"))
        want = before.astype(np.float64) * (1 - lr * wd) - lr * (mh / (1 - b1 ** t)) / (np.sqrt(vh / (1 - b2 ** t)) + eps)
        assert np.abs(th - want).max() <= 1e-7 * np.abs(want).max()


def test_init_state_is_zero(O):
    for bm, bv in [(16, 16), (8, 4), (2, 3), (32, 32)]:
        n = 1000
        st = O.new_state(n, 256, bm, bv)
        if bm != 32:
            assert (O.unpack(st.m_codes, n, bm) == (1 << (bm - 1))).all()
            assert (O.unpack(st.v_codes, n, bv) == 0).all()
            assert (st.m_scales == 0).all() and (st.v_scales == 0).all()
        assert (O.dequantize(st.m_codes, st.m_scales, n, bm, 256, O.LINEAR) == 0).all()
        assert (O.dequantize(st.v_codes, st.v_scales, n, bv, 256, O.LOG) == 0).all()


def test_width_change_inside_a_step_equals_step_at_new_width(O):
    """Stored at (8,4), written at (4,8): same as quantizing the fresh moments at the new widths."""
    rng = np.random.default_rng(6)
    n = 128 * 9 + 3
    th = rng.normal(0, 0.02, n).astype(np.float32)
    st = O.new_state(n, 128, 8, 4)
    g1 = (rng.standard_t(4, n) * 1e-3).astype(np.float32)
    st, _ = O.step(th, g1, st, 128, t=1, **HP)
    g2 = (rng.standard_t(4, n) * 1e-3).astype(np.float32)
    th_a = th.copy()
    st_a, _ = O.step(th_a, g2, st, 128, t=2, bits_m_out=4, bits_v_out=8, **HP)
    # the same moments by hand
    mh = O.dequantize(st.m_codes, st.m_scales, n, 8, 128, O.LINEAR)
    vh = O.dequantize(st.v_codes, st.v_scales, n, 4, 128, O.LOG)
    b1, b2 = np.float32(0.9), np.float32(0.999)
    m = np.array([_fma32(float(b1), float(a), float(c)) for a, c in zip(mh, np.float32(1 - 0.9) * g2)], np.float32)
    v = np.array([_fma32(float(b2), float(a), float(c))
                  for a, c in zip(vh, (np.float32(1 - 0.999) * g2) * g2)], np.float32)
    cm, sm = O.quantize(m, 4, 128, O.LINEAR)
    cv, sv = O.quantize(v, 8, 128, O.LOG)
    assert (cm == st_a.m_codes).all() and (sm == st_a.m_scales).all()
    assert (cv == st_a.v_codes).all() and (sv == st_a.v_scales).all()


def test_bf16_grads_widen_exactly(O):
    rng = np.random.default_rng(7)
    n = 1024
    g32 = (rng.standard_t(3, n) * 1e-3).astype(np.float32)
    gb = torch.from_numpy(g32).to(torch.bfloat16)
    bits16 = gb.view(torch.int16).numpy().view(np.uint16).copy()
    widened = gb.to(torch.float32).numpy()
    th1 = rng.normal(0, 0.02, n).astype(np.float32)
    th2 = th1.copy()
    st1 = O.new_state(n, 128, 8, 4)
    st2 = O.new_state(n, 128, 8, 4)
    st1, s1 = O.step(th1, bits16, st1, 128, t=1, want_stats=True, **HP)
    st2, s2 = O.step(th2, widened, st2, 128, t=1, want_stats=True, **HP)
    assert (th1 == th2).all() and (st1.m_codes == st2.m_codes).all() and (st1.v_codes == st2.v_codes).all()
    assert (s1 == s2).all()


def test_half_precision_conversions_match_the_library(O):
    """fp16 widening and the nearest-even roundings to bf16 / fp16 against torch's conversions."""
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 1, 100000) * 10.0 ** rng.uniform(-9, 5, 100000),
                        [0, -0.0, 65504, 65519.9, 65520, 6.1e-5, 5.96e-8, 2.98e-8, 2.99e-8, 1e-10, -3e-8]]).astype(np.float32)
    t = torch.from_numpy(x)
    assert (O.round_lp(x, "bf16") == t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)).all()
    assert (O.round_lp(x, "fp16") == t.to(torch.float16).view(torch.int16).numpy().view(np.uint16)).all()
    allh = np.arange(65536, dtype=np.uint16)
    want = torch.from_numpy(allh.view(np.int16)).view(torch.float16).float().numpy()
    got = O.widen_f16(allh)
    fin = np.isfinite(want)
    assert (got[fin].view(np.uint32) == want[fin].view(np.uint32)).all()


def test_loss_scale_and_skipped_step(O):
    """Gradients scaled by S and multiplied back by 1/S (a power of two) give the unscaled step bit for
    bit; a step with found_inf leaves everything untouched."""
    rng = np.random.default_rng(9)
    n = 128 * 3 + 17
    g = (rng.standard_t(4, n) * 1e-3).astype(np.float32)
    th1 = rng.normal(0, 0.02, n).astype(np.float32)
    th2 = th1.copy()
    st1, _ = O.step(th1, g, O.new_state(n, 128, 8, 4), 128, t=1, **HP)
    st2, _ = O.step(th2, (g * np.float32(1024)).astype(np.float32), O.new_state(n, 128, 8, 4), 128, t=1,
                    inv_grad_scale=1.0 / 1024, **HP)
    assert (th1 == th2).all() and (st1.m_codes == st2.m_codes).all() and (st1.v_codes == st2.v_codes).all()
    before = th1.copy()
    st3, _ = O.step(th1, g, st1, 128, t=2, found_inf=True, **HP)
    assert (th1 == before).all() and st3 is st1


@pytest.mark.parametrize("bits_m,bits_v,v_mode", [(4, 8, "log"), (3, 16, "pl"), (32, 4, "log"), (8, 32, "log"), (2, 2, "log"),
                                                  (4, 4, "sr"), (8, 16, "sr"), (4, 3, "ts"), (16, 8, "ts")])
def test_a_tensor_stepped_range_by_range_equals_the_tensor_stepped_whole(O, bits_m, bits_v, v_mode):
    """Blocks are independent given their inputs: stepping block-aligned ranges one by one (as the full-size
    GPU tests do, over a thread pool) writes the same bytes as one call over the tensor, ragged tail included."""
    rng = np.random.RandomState(7)
    n, block = 128 * 37 + 55, 128
    vm = {"pl": O.LOG_PL, "sr": O.LOG_SR, "ts": O.LOG_TS}.get(v_mode, O.LOG)
    th = (rng.randn(n) * 0.02).astype(np.float32)
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01, sr_seed=0xABCDEF0123, tensor_index=7)
    whole_t, parts_t = th.copy(), th.copy()
    whole = parts = O.new_state(n, block, bits_m, bits_v, vm)
    for t in (1, 2, 3):
        g = (rng.standard_t(4, n) * 1e-3).astype(np.float32)
        whole, stats = O.step(whole_t, g, whole, block, t=t, want_stats=True, v_mode=vm, **hp)
        mc, ms = O.alloc_state(n, bits_m, block)
        vc, vs = O.alloc_state(n, bits_v, block, vm)
        nxt = O.State(mc, ms, bits_m, vc, vs, bits_v)
        total = np.zeros(4)
        for e0 in reversed(range(0, n, block * 10)):          # any order
            s4 = np.zeros(4)
            O.step_range(parts_t, g, e0, min(n, e0 + block * 10), block, parts, nxt, t=t, v_mode=vm, stats=s4, **hp)
            total += s4
        parts = nxt
        assert (whole_t == parts_t).all()
        assert (whole.m_codes == parts.m_codes).all() and (whole.v_codes == parts.v_codes).all()
        assert (whole.m_scales.view(np.uint32) == parts.m_scales.view(np.uint32)).all()
        assert (whole.v_scales.view(np.uint32) == parts.v_scales.view(np.uint32)).all()
        np.testing.assert_allclose(total, stats, rtol=1e-12)

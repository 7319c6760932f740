"""Pins of the "pl" variant of the log quantizer (the logarithm replaced by the piecewise-linear one
that the fp32 bit pattern is).  None of the checks below restates the oracle's arithmetic: they use
exact integer arithmetic on bit patterns, closed forms at powers of two, and the analytic bound that
links the piecewise-linear logarithm to log2."""
import numpy as np
import pytest


def _bits(x):
    return np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.int64)


def _heavy(rng, n, scale=1e-3):
    return (rng.standard_t(3, n) * scale).astype(np.float32)


def test_pl_is_log2_at_powers_of_two_and_linear_between():
    # what the variant rests on: bits(x) * 2^-23 - 127 equals log2 at powers of two and lies below
    # log2 by at most 0.0861 between them (the maximum of log2(1 + t) - t, at t = 1/ln2 - 1)
    x = np.exp2(np.arange(-100, 30)).astype(np.float32)
    assert (_bits(x) * 2.0 ** -23 - 127 == np.log2(x.astype(np.float64))).all()
    t = np.linspace(0, 1, 100001)
    gap = np.log2(1 + t) - t
    assert gap.min() >= -1e-15 and gap.max() <= 0.0861
    y = (1 + t[:-1]).astype(np.float32)
    np.testing.assert_allclose(_bits(y) * 2.0 ** -23 - 127, y.astype(np.float64) - 1, atol=1e-7)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_octave_widths_are_the_same_code_in_both_variants(O, bits):
    rng = np.random.default_rng(bits)
    x = (_heavy(rng, 128 * 30 + 5) ** 2).astype(np.float32)
    a, sa = O.quantize(x, bits, 128, O.LOG)
    b, sb = O.quantize(x, bits, 128, O.LOG_PL)
    assert (a == b).all() and (sa == sb).all()
    assert (O.dequantize(a, sa, x.size, bits, 128, O.LOG) == O.dequantize(b, sb, x.size, bits, 128, O.LOG_PL)).all()


@pytest.mark.parametrize("bits", [8, 16])
def test_codes_at_powers_of_two_below_the_maximum(O, bits):
    # x = s * 2^-k sits exactly k octaves below the maximum in either logarithm: the code is
    # K - k*K/R whenever that is an integer, and such a code decodes to x exactly
    K, R = (1 << bits) - 1, 30
    for s in (1.0, 3.0e-7, 1.7):
        ks = np.arange(0, R + 1)
        x = (np.float32(s) * np.exp2(-ks)).astype(np.float32)
        blk = np.full(128, x[-1], np.float32)
        blk[:ks.size] = x
        c, sc = O.quantize(blk, bits, 128, O.LOG_PL)
        assert sc[0] == np.float32(s)
        codes = O.unpack(c, 128, bits)[:ks.size].astype(np.int64)
        whole = (ks * K) % R == 0
        assert (codes[whole] == K - ks[whole] * K // R).all()
        assert (np.abs(codes - (K - ks * K / R)) <= 0.5).all()
        xh = O.dequantize(c, sc, 128, bits, 128, O.LOG_PL)[:ks.size].astype(np.float64)
        assert (xh[whole] == x[whole].astype(np.float64)).all()
        assert xh[0] == np.float32(s)            # the block maximum comes back exactly


@pytest.mark.parametrize("bits", [8, 16])
def test_code_is_the_nearest_level_in_bit_pattern_distance(O, bits):
    """Brute force with exact integers: among all 2^b decodable levels of the block, the chosen one
    is nearest to x in bit-pattern distance (= distance in the piecewise-linear logarithm)."""
    rng = np.random.default_rng(50 + bits)
    K = (1 << bits) - 1
    n = 128
    for trial in range(4):
        x = (_heavy(rng, n, 1e-3 * 10.0 ** -trial) ** 2).astype(np.float32)
        x[3] = 0.0
        c, s = O.quantize(x, bits, 128, O.LOG_PL)
        codes = O.unpack(c, n, bits).astype(np.int64)
        # every level of this block: decode all codes against the same scale
        all_codes = np.arange(K + 1, dtype=np.uint32)
        levels = np.concatenate([
            O.dequantize(O.pack(np.resize(all_codes[i:i + 128], 128), bits), s, 128, bits, 128, O.LOG_PL)
            for i in range(0, K + 1, 128)])[:K + 1]
        lb = _bits(levels)
        assert (np.diff(lb) > 0).all()                      # levels increase with the code
        xb = _bits(x)
        best = np.abs(xb[:, None] - lb[None, :]).min(axis=1)
        got = np.abs(xb - lb[codes])
        # slack: a level sits within half a unit of the pattern of its ideal place j*D/K and the
        # code boundary is exactly half-way between ideal places
        assert (got <= best + 1).all(), int((got - best).max())
        floor_bits = lb[0]
        assert (codes[xb <= floor_bits] == 0).all()


@pytest.mark.parametrize("bits", [8, 16])
def test_error_bound_in_octaves(O, bits):
    # half a code step in the piecewise-linear logarithm, stretched by the largest slope ratio between
    # it and log2 (d log2 / d pl = 1/((1+t) ln 2) <= 1/ln 2 = 1.4427): |log2(x^/x)| <= 0.7214 * R/K
    rng = np.random.default_rng(60 + bits)
    n = 128 * 150 + 9
    K, R = (1 << bits) - 1, 30
    x = (_heavy(rng, n) ** 2).astype(np.float32)
    c, s = O.quantize(x, bits, 128, O.LOG_PL)
    xh = O.dequantize(c, s, n, bits, 128, O.LOG_PL).astype(np.float64)
    sx = np.repeat(s, 128)[:n].astype(np.float64)
    inr = x.astype(np.float64) >= sx * 2.0 ** -R
    err = np.abs(np.log2(xh[inr] / x[inr].astype(np.float64)))
    assert err.max() <= 0.7214 * R / K * 1.01
    assert err.max() >= 0.5 * R / K * 0.9               # and it is a quantizer of that resolution, not finer
    codes = O.unpack(c, n, bits).astype(np.int64)
    assert (xh[codes == K] == sx[codes == K]).all()
    pad = np.zeros(s.size * 128, np.float32)
    pad[:n] = x
    assert (pad.reshape(-1, 128).max(1) == s).all()


@pytest.mark.parametrize("bits", [8, 16])
def test_idempotent_monotone_and_zero_blocks(O, bits):
    rng = np.random.default_rng(70 + bits)
    n = 128 * 20
    x = (_heavy(rng, n) ** 2).astype(np.float32)
    x[128:256] = 0.0                                     # a zero block
    x[256:384] = np.float32(1e-38)                       # a block below the tiny-scale rule
    c, s = O.quantize(x, bits, 128, O.LOG_PL)
    assert s[1] == 0 and s[2] == 0
    xh = O.dequantize(c, s, n, bits, 128, O.LOG_PL)
    assert (xh[128:384] == 0).all()
    c2, s2 = O.quantize(xh, bits, 128, O.LOG_PL)
    assert (c2 == c).all() and (s2 == s).all()
    # a larger value never gets a smaller code
    y = np.exp2(np.linspace(-35, 0, 128 * 40)).astype(np.float32).reshape(40, 128)
    y[:, -1] = 1.0
    cy, _ = O.quantize(y.ravel(), bits, 128, O.LOG_PL)
    codes = O.unpack(cy, y.size, bits).reshape(40, 128)[:, :-1].ravel().astype(np.int64)
    assert (np.diff(codes) >= 0).all()
    # repack to the same width is the identity; scales survive a change of width
    for b2 in (4, 8, 16):
        c3, s3 = O.repack(c, s, bits, b2, n, 128, O.LOG_PL)
        assert (s3 == s).all()
        if b2 == bits:
            assert (c3 == c).all()


def test_sixteen_bit_pl_states_track_textbook_adamw(O):
    from test_oracle_adamw import HP, textbook_adamw
    rng = np.random.default_rng(3)
    n = 512
    theta0 = rng.normal(0, 0.02, n).astype(np.float32)
    grads = [(rng.choice([-1.0, 1.0], n) * 1e-3 * rng.uniform(0.05, 1.0, n)).astype(np.float32) for _ in range(10)]
    th = theta0.copy()
    st = O.new_state(n, 128, 16, 16)
    for t, g in enumerate(grads, start=1):
        st, _ = O.step(th, g, st, 128, t=t, v_mode=O.LOG_PL, **HP)
        ref, _, _ = textbook_adamw(theta0, grads[:t], **HP)
        lim = 1e-3 if t == 1 else 5e-3
        assert np.abs(th - ref).max() <= lim * HP["lr"], (t, np.abs(th - ref).max() / HP["lr"])


def test_step_uses_the_variant_for_the_second_moment_only(O):
    from test_oracle_adamw import HP
    rng = np.random.default_rng(9)
    n = 128 * 3 + 11
    th_a = rng.normal(0, 0.02, n).astype(np.float32)
    th_b = th_a.copy()
    g = (_heavy(rng, n)).astype(np.float32)
    sa, _ = O.step(th_a, g, O.new_state(n, 128, 8, 8), 128, t=1, **HP)
    sb, _ = O.step(th_b, g, O.new_state(n, 128, 8, 8), 128, t=1, v_mode=O.LOG_PL, **HP)
    assert (sa.m_codes == sb.m_codes).all() and (sa.m_scales == sb.m_scales).all()
    assert (sa.v_scales == sb.v_scales).all() and (sa.v_codes != sb.v_codes).any()
    vh = O.dequantize(sb.v_codes, sb.v_scales, n, 8, 128, O.LOG_PL).astype(np.float64)
    mh = O.dequantize(sb.m_codes, sb.m_scales, n, 8, 128, O.LINEAR).astype(np.float64)
    lr, wd, eps, b1, b2 = (HP[k] for k in ("lr", "weight_decay", "eps", "beta1", "beta2"))
    # theta from the decoded new codes of the variant
    before = np.random.default_rng(9).normal(0, 0.02, n).astype(np.float32).astype(np.float64)
    want = before * (1 - lr * wd) - lr * (mh / (1 - b1)) / (np.sqrt(vh / (1 - b2)) + eps)
    assert np.abs(th_b - want).max() <= 1e-7 * np.abs(want).max()


@pytest.mark.parametrize("bits", [8, 16])
def test_decode_levels_are_the_rounded_rational_distance(O, bits):
    """Every level against exact rational arithmetic: code K - j sits round(j * 30 * 2^23 / K) units of
    the bit pattern below the scale.  At 8 bits that holds for all codes; at 16 bits the 32-bit
    multiplier of the definition lands one unit off for a few codes whose exact distance is within
    a hair of a half, and nowhere else."""
    from fractions import Fraction
    import math
    K, D = (1 << bits) - 1, 30 << 23
    s = np.array([1.5], dtype=np.float32)
    codes = np.arange(K + 1, dtype=np.uint32)
    levels = np.concatenate([
        O.dequantize(O.pack(np.resize(codes[i:i + 128], 128), bits), s, 128, bits, 128, O.LOG_PL)
        for i in range(0, K + 1, 128)])[:K + 1]
    below = int(_bits(s)[0]) - _bits(levels)
    want = np.array([math.floor(Fraction((K - int(c)) * D, K) + Fraction(1, 2)) for c in codes], dtype=np.int64)
    diff = below - want
    assert np.abs(diff).max() <= 1
    if bits == 8:
        assert (diff == 0).all()
    else:
        off = np.flatnonzero(diff)
        assert off.size <= 200
        frac = np.array([float(Fraction((K - int(codes[i])) * D, K) % 1) for i in off])
        assert (np.abs(frac - 0.5) < 0.02).all()

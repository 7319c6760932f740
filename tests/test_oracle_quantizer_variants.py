"""Pins of the two further readings of "logarithmic quantization" (Sec. 3.5 names the mode, no formula):
variant "sr" (stochastic rounding on the piecewise-linear logarithm of x / block maximum) and variant "ts"
(two scales per block: the codes span the block's own minimum..maximum).

Nothing below restates the oracle's arithmetic.  The generator is pinned by an independently written
inverse (it is a bijection) and by the independence of its outputs; the stochastic rounding by exact
enumeration over all 2^32 random words and exact rational arithmetic on the levels; the two-scale code by
hand-worked examples (tests/golden), exact end points and the analytic error bound."""
from fractions import Fraction

import numpy as np
import pytest

M32 = 0xFFFFFFFF
ONE_BITS = 0x3F800000


def _f(x):
    return float(np.float32(x))


def _bits(x):
    return int(np.float32(x).view(np.uint32))


def _heavy_v(rng, n, scale=1e-3):
    return ((rng.standard_t(3, n) * scale) ** 2).astype(np.float32)


# ---- the generator ---------------------------------------------------------------------------------------------
def _unmix32(h):
    """Inverse of the mixing function, written from its description step by step, last step first."""
    h ^= h >> 16
    h = (h * pow(0xC2B2AE35, -1, 1 << 32)) & M32
    h ^= (h >> 13) ^ (h >> 26)
    h = (h * pow(0x85EBCA6B, -1, 1 << 32)) & M32
    h ^= h >> 16
    return h


def test_the_mixing_function_is_a_bijection_and_mixes(O):
    rng = np.random.default_rng(0)
    words = [0, 1, 2, M32, 0x80000000, 0x9E3779B9] + [int(x) for x in rng.integers(0, 1 << 32, 5000)]
    for h in words:
        assert _unmix32(O.mix32(h)) == h
    assert O.mix32(0) == 0                                    # the one fixed point every xor-shift/multiply chain has
    # avalanche: flipping one input bit flips about half of the output bits
    flips = [bin(O.mix32(h) ^ O.mix32(h ^ (1 << int(b)))).count("1")
             for h, b in zip(words[6:2006], rng.integers(0, 32, 2000))]
    assert 15.0 < np.mean(flips) < 17.0 and min(flips) >= 4


def test_key_and_words_depend_on_seed_step_tensor_and_element(O):
    base = O.sr_key(0x1234567890ABCDEF, 7, 3)
    others = {O.sr_key(0x1234567890ABCDEF ^ 1, 7, 3), O.sr_key(0x1234567890ABCDEF ^ (1 << 40), 7, 3),
              O.sr_key(0x1234567890ABCDEF, 8, 3), O.sr_key(0x1234567890ABCDEF, 7 + (1 << 33), 3),
              O.sr_key(0x1234567890ABCDEF, 7, 4)}
    assert base not in others and len(others) == 5
    # for a fixed key the low word of the element index maps one-to-one to the random word
    w = [O.sr_word(base, e) for e in range(1 << 16)]
    assert len(set(w)) == 1 << 16
    assert O.sr_word(base, 5) != O.sr_word(base, 5 + (1 << 32))     # elements beyond 2^32 draw from another stream
    assert O.sr_word(base, 5) != O.sr_word(base ^ 1, 5)
    # uniform enough for rounding: the mean of 65536 consecutive words sits at 2^31 within 4 standard errors
    assert abs(np.mean(w) / 2.0 ** 32 - 0.5) < 4 * (1 / np.sqrt(12 * len(w)))


# ---- stochastic rounding -----------------------------------------------------------------------------------------
def _expected_level(O, x, s, bits):
    """E[y^] over all 2^32 random words as an exact rational, from the exact enumeration."""
    (c_lo, n_lo), (c_hi, n_hi) = O.sr_enumerate(x, s, bits)
    assert n_lo + n_hi == 1 << 32 and abs(c_hi - c_lo) <= 1
    return (Fraction(O.sr_level(c_lo, bits)) * n_lo + Fraction(O.sr_level(c_hi, bits)) * n_hi) / (1 << 32), (c_lo, c_hi)


def _y(x, s):
    """The normalised value the variant rounds: fl(x * fl(fl(1/s) * (1 + 2^-21))), in fp32 steps."""
    rs = np.float32(1.0) / np.float32(s)
    c1 = np.float32(rs * np.float32(1 + 2.0 ** -21))
    return float(np.float32(np.float32(x) * c1))


LG_LEVELS = {2: 0, 3: 0, 4: 0, 8: 3, 16: 11}      # levels per octave: 1, 1, 1, 8, 2048


@pytest.mark.parametrize("bits,x,s", [(2, 0.3, 1.0), (4, 0.0123, 0.771), (8, 2.9e-7, 1.7e-6), (16, 0.61, 1.3)])
def test_exact_enumeration_is_unbiased(O, bits, x, s):
    """Every one of the 2^32 random words, counted: the expectation of the decoded level equals the value
    that was rounded, as an exact rational (no power of two lies between two neighbouring levels, and
    between powers of two the bit pattern is linear in the value)."""
    e, (c_lo, c_hi) = _expected_level(O, x, s, bits)
    assert c_hi == c_lo + 1
    assert e == Fraction(_y(x, s))
    assert abs(float(e) * _f(s) / _f(x) - 1) < 1e-6            # and y * s is x to rounding


def test_rounding_threshold_in_closed_form_and_unbiased_everywhere(O):
    """The count of words that round down needs no enumeration: with n the distance below 1.0 in units of the
    bit pattern, the code drops exactly when the low 32 bits of n << (9 + g) carry.  Checked at the threshold
    word for many values at every width (the enumeration above validates the closed form itself), and the
    expectation that follows from the counts equals the rounded value exactly."""
    rng = np.random.default_rng(1)
    for bits in (2, 3, 4, 8, 16):
        K, g = (1 << bits) - 1, LG_LEVELS[bits]
        octaves = K / (1 << g)
        for _ in range(400):
            s = _f(10.0 ** rng.uniform(-12, 3))
            x = _f(s * 2.0 ** -rng.uniform(0, octaves * 0.98))
            y = _y(x, s)
            n = min(max(ONE_BITS - _bits(y), 0), K << (23 - g))
            j0, low = divmod(n << (9 + g), 1 << 32)
            if j0 >= K:
                continue
            assert O.sr_code(x, s, bits, 0) == K - j0
            if low == 0:
                assert O.sr_code(x, s, bits, M32) == K - j0        # on a level: it stays there whatever the word
                continue
            thr = (1 << 32) - low                       # first word that carries
            assert O.sr_code(x, s, bits, thr - 1) == K - j0
            assert O.sr_code(x, s, bits, thr) == K - j0 - 1 and O.sr_code(x, s, bits, M32) == K - j0 - 1
            hi, lo = Fraction(O.sr_level(K - j0, bits)), Fraction(O.sr_level(K - j0 - 1, bits))
            assert (hi * ((1 << 32) - low) + lo * low) / (1 << 32) == Fraction(y)


@pytest.mark.parametrize("bits", [2, 3, 4, 8, 16])
def test_maximum_floor_zero_block_and_monotone_in_the_word(O, bits):
    K = (1 << bits) - 1
    rng = np.random.default_rng(bits)
    for s in (1.0, 3.1e-7, 0.999999, 1.7, 2.0 ** -90):
        for U in (0, 1, 0x7FFFFFFF, 0x80000000, M32):
            assert O.sr_code(s, s, bits, U) == K                 # the block maximum is code K whatever the word
            assert O.sr_code(0.0, s, bits, U) == 0               # zero: the floor level
            assert O.sr_code(_f(s * 2.0 ** -40), s, bits, U) == 0
        x = _f(s * 2.0 ** -rng.uniform(0.2, K / (1 << LG_LEVELS[bits]) - 0.5))
        codes = [O.sr_code(x, s, bits, U) for U in np.linspace(0, M32, 257).astype(np.uint64)]
        assert all(a >= b for a, b in zip(codes, codes[1:])) and codes[0] - codes[-1] <= 1
    # scales whose reciprocal rounds down, so that s * fl(1/s) falls just short of 1: still code K, for every word
    short = [s for s in (_f(t) for t in rng.uniform(1.0, 2.0, 4000))
             if float(np.float32(np.float32(s) * (np.float32(1.0) / np.float32(s)))) < 1.0]
    assert len(short) > 100
    for s in short[:200]:
        assert O.sr_code(s, s, bits, M32) == K and O.sr_code(s, s, bits, 0) == K
    assert O.sr_level(K, bits) == 1.0                            # so the maximum decodes to the scale exactly
    octaves = K / (1 << LG_LEVELS[bits])                         # 3, 7, 15, 31.875, 32 (- 1/2048)
    whole = int(np.ceil(octaves))
    assert O.sr_level(0, bits) == 2.0 ** -whole * (1 + (whole - octaves))     # linear inside the last octave
    v = np.zeros(256, np.float32)
    v[128:] = 2.0 ** -110                                        # below the tiny rule: an all-zero block as well
    c, sc = O.quantize(v, bits, 128, O.LOG_SR, key=9)
    assert (sc == 0).all() and (O.unpack(c, 256, bits) == 0).all()
    assert (O.dequantize(c, sc, 256, bits, 128, O.LOG_SR) == 0).all()


@pytest.mark.parametrize("bits", [2, 3, 4, 8, 16])
def test_a_tensor_uses_the_word_of_each_element_and_decodes_between_neighbours(O, bits):
    rng = np.random.default_rng(10 + bits)
    n, block, key = 128 * 9 + 77, 128, O.sr_key(42, 3, 5)
    v = _heavy_v(rng, n)
    c, sc = O.quantize(v, bits, block, O.LOG_SR, key=key)
    codes = O.unpack(c, n, bits)
    K = (1 << bits) - 1
    for i in rng.integers(0, n, 300):
        i = int(i)
        assert codes[i] == O.sr_code(v[i], sc[i // block], bits, O.sr_word(key, i))
    d = O.dequantize(c, sc, n, bits, block, O.LOG_SR)
    s_el = np.repeat(sc, block)[:n].astype(np.float64)
    step = 1.0 / (1 << LG_LEVELS[bits])
    floor = s_el * O.sr_level(0, bits)
    inside = v > floor * 1.0000001
    # the decoded value is one of the two levels around x: within the widest gap between neighbouring
    # levels, log2(1 + 1/L) octaves (the levels are evenly spaced in the mantissa, not in log2)
    step = np.log2(1 + step)
    assert (np.abs(np.log2(d[inside].astype(np.float64) / v[inside])) <= step * 1.0000001 + 1e-6).all()
    assert (d[~inside] == floor[~inside].astype(np.float32)).all()
    for b0 in range(0, n, block):
        assert d[b0:b0 + block].max() == sc[b0 // block]
    # another key, other codes; the same key, the same codes
    c2, _ = O.quantize(v, bits, block, O.LOG_SR, key=key ^ 1)
    c3, _ = O.quantize(v, bits, block, O.LOG_SR, key=key)
    assert (c3 == c).all() and (c2 != c).any()


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_the_mean_over_keys_approaches_the_value(O, bits):
    """Through the tensor path: averaged over many keys the decoded values converge on the inputs (above the
    floor), which round-to-nearest codes do not do."""
    rng = np.random.default_rng(3)
    n, block = 1024, 128
    v = _heavy_v(rng, n)
    K = (1 << bits) - 1
    acc = np.zeros(n)
    reps = 400
    for k in range(reps):
        c, sc = O.quantize(v, bits, block, O.LOG_SR, key=O.sr_key(k, 1, 0))
        acc += O.dequantize(c, sc, n, bits, block, O.LOG_SR)
    mean = acc / reps
    s_el = np.repeat(sc, block).astype(np.float64)
    step = 1.0 / (1 << LG_LEVELS[bits])
    inside = v > s_el * O.sr_level(0, bits) * 1.01
    rel = mean[inside] / v[inside] - 1
    # a two-point distribution between neighbouring levels a ratio 2^step apart: relative spread at most (2^step - 1) / 2
    sigma = (2.0 ** step - 1) / 2 / np.sqrt(reps)
    assert np.abs(rel).max() < 5 * sigma + 3e-3
    assert abs(rel.mean()) < 5 * sigma / np.sqrt(inside.sum()) + 1e-3
    det_c, det_s = O.quantize(v, bits, block, O.LOG)
    det = O.dequantize(det_c, det_s, n, bits, block, O.LOG)[inside] / v[inside] - 1
    if bits <= 4:
        assert np.abs(det).mean() > 5 * np.abs(rel).mean()       # rounding to nearest keeps its per-element error


@pytest.mark.parametrize("bits", [2, 3, 4, 8, 16])
def test_keyless_requantization_rounds_to_nearest_and_returns_the_same_codes(O, bits):
    """A re-pack has no step to draw words from: the variant then rounds to nearest, and a stored state goes
    back to itself (the scale is reproduced by the maximum, every level lands on itself)."""
    rng = np.random.default_rng(20 + bits)
    n, block = 128 * 6 + 19, 128
    v = _heavy_v(rng, n)
    c, sc = O.quantize(v, bits, block, O.LOG_SR, key=77)
    c2, sc2 = O.repack(c, sc, bits, bits, n, block, O.LOG_SR)
    assert (c2 == c).all() and (sc2.view(np.uint32) == sc.view(np.uint32)).all()
    for wide in (b for b in (4, 8, 16) if b > bits):
        cw, sw = O.repack(c, sc, bits, wide, n, block, O.LOG_SR)
        cb, sb = O.repack(cw, sw, wide, bits, n, block, O.LOG_SR)
        assert (sw.view(np.uint32) == sc.view(np.uint32)).all()
        assert (cb == c).all(), (bits, wide)


def test_adamw_with_stochastic_rounding_follows_textbook_adamw_at_16_bits(O):
    rng = np.random.default_rng(5)
    n, block = 1024, 128
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    th = (rng.normal(0, 0.02, n)).astype(np.float32)
    ref, m, v = th.astype(np.float64), np.zeros(n), np.zeros(n)
    st = O.new_state(n, block, 16, 16, O.LOG_SR)
    for t in range(1, 11):
        g = (rng.choice([-1.0, 1.0], n) * 1e-3 * rng.uniform(0.05, 1.0, n)).astype(np.float32)
        st, _ = O.step(th, g, st, block, t=t, v_mode=O.LOG_SR, sr_seed=99, tensor_index=2, **hp)
        gd = g.astype(np.float64)
        m = 0.9 * m + 0.1 * gd
        v = 0.999 * v + 0.001 * gd * gd
        ref = ref * (1 - 1e-3 * 0.01) - 1e-3 * (m / (1 - 0.9 ** t)) / (np.sqrt(v / (1 - 0.999 ** t)) + 1e-8)
    assert np.abs(th - ref).max() <= 5e-3 * 1e-3
    # the seed matters and is reproducible
    th_a, th_b, th_c = (rng.normal(0, 0.02, n).astype(np.float32),) * 3
    outs = []
    for seed in (1, 1, 2):
        s0 = O.new_state(n, block, 4, 4, O.LOG_SR)
        s1, _ = O.step(th_a.copy(), g, s0, block, t=1, v_mode=O.LOG_SR, sr_seed=seed, tensor_index=0, **hp)
        outs.append(s1.v_codes.copy())
    assert (outs[0] == outs[1]).all() and (outs[0] != outs[2]).any()


# ---- two scales per block ------------------------------------------------------------------------------------------
def _golden_ts():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "quant_worked_examples.txt")
    for line in open(path):
        if line.startswith("ts "):
            head, xs, codes, dec = [p.strip() for p in line.split("|")]
            _, bits, hi, lo = head.split()
            yield (int(bits), float(hi), float(lo), [float(t) for t in xs.split()], [int(t) for t in codes.split()],
                   [float(t) for t in dec.split()])


def test_two_scale_worked_examples(O):
    cases = list(_golden_ts())
    assert len(cases) >= 4
    for bits, hi, lo, xs, codes, dec in cases:
        x = np.array(xs, dtype=np.float32)
        c, sc = O.quantize(x, bits, len(xs), O.LOG_TS)
        assert sc.tolist() == [np.float32(hi), np.float32(lo)], (bits, sc)
        assert O.unpack(c, len(xs), bits).tolist() == codes, (bits, O.unpack(c, len(xs), bits))
        np.testing.assert_allclose(O.dequantize(c, sc, len(xs), bits, len(xs), O.LOG_TS), dec, rtol=1e-6)


@pytest.mark.parametrize("bits", [2, 3, 4, 8, 16])
def test_two_scale_end_points_error_bound_and_monotone_codes(O, bits):
    rng = np.random.default_rng(30 + bits)
    block, nb = 128, 40
    K = (1 << bits) - 1
    v = _heavy_v(rng, block * nb)
    v[5 * block:6 * block] = np.float32(3.3e-9)                   # a block of equal values
    v[7 * block] = 0.0                                            # a zero element among ordinary ones
    v[9 * block:10 * block] = 0.0                                 # a zero block
    c, sc = O.quantize(v, bits, block, O.LOG_TS)
    assert sc.size == 2 * nb
    codes = O.unpack(c, v.size, bits).reshape(nb, block)
    d = O.dequantize(c, sc, v.size, bits, block, O.LOG_TS).reshape(nb, block)
    x = v.reshape(nb, block)
    for k in range(nb):
        hi, lo = sc[2 * k], sc[2 * k + 1]
        if k == 9:
            assert hi == 0 and lo == 0 and (codes[k] == 0).all() and (d[k] == 0).all()
            continue
        assert hi == x[k].max() and lo == max(x[k].min(), np.float32(hi * np.float32(2.0 ** -30)))
        assert d[k].max() == hi and d[k].min() == lo              # both end points are reproduced exactly
        assert codes[k][np.argmax(x[k])] == K
        if k == 5:
            assert (codes[k] == K).all() and (d[k] == hi).all()
            continue
        assert codes[k][np.argmin(x[k])] == 0
        W = min(np.log2(float(hi) / float(lo)), 30.0)
        inside = x[k] >= lo
        err = np.abs(np.log2(d[k][inside].astype(np.float64) / x[k][inside]))
        assert err.max() <= W / (2 * K) * 1.00001 + 1.2e-5        # half a code step, plus the polynomials
        order = np.argsort(x[k], kind="stable")
        assert (np.diff(codes[k][order].astype(np.int64)) >= 0).all()
    assert codes[7][0] == 0 and d[7][0] == sc[15]                 # the zero element sits at the floor, not at zero


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_two_scale_is_idempotent_and_adapts_to_the_range(O, bits):
    rng = np.random.default_rng(40 + bits)
    n, block = 128 * 12, 128
    v = _heavy_v(rng, n)
    c, sc = O.quantize(v, bits, block, O.LOG_TS)
    d = O.dequantize(c, sc, n, bits, block, O.LOG_TS)
    c2, sc2 = O.quantize(d, bits, block, O.LOG_TS)
    assert (sc2.view(np.uint32) == sc.view(np.uint32)).all()
    assert (c2 == c).all()
    # a block that spans few octaves is coded finer than the fixed-range code of the same width, one that
    # spans more than the fixed range keeps its small elements instead of flooring them
    K = (1 << bits) - 1
    narrow = (np.float32(1e-6) * np.exp2(-rng.uniform(0, 1.5, block))).astype(np.float32)
    e_ts = np.abs(np.log2(O.dequantize(*O.quantize(narrow, bits, block, O.LOG_TS), block, bits, block, O.LOG_TS) / narrow)).max()
    e_fx = np.abs(np.log2(O.dequantize(*O.quantize(narrow, bits, block, O.LOG), block, bits, block, O.LOG) / narrow)).max()
    assert e_ts <= 1.5 / (2 * K) * 1.001 + 1.2e-5 and e_ts < 0.6 * e_fx


def test_two_scale_adamw_follows_textbook_adamw_at_16_bits_and_repack_keeps_both_scales(O):
    rng = np.random.default_rng(6)
    n, block = 1024, 128
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    th = (rng.normal(0, 0.02, n)).astype(np.float32)
    ref, m, v = th.astype(np.float64), np.zeros(n), np.zeros(n)
    st = O.new_state(n, block, 16, 16, O.LOG_TS)
    assert st.v_scales.size == 2 * (n // block)
    for t in range(1, 11):
        g = (rng.choice([-1.0, 1.0], n) * 1e-3 * rng.uniform(0.05, 1.0, n)).astype(np.float32)
        st, _ = O.step(th, g, st, block, t=t, v_mode=O.LOG_TS, **hp)
        gd = g.astype(np.float64)
        m = 0.9 * m + 0.1 * gd
        v = 0.999 * v + 0.001 * gd * gd
        ref = ref * (1 - 1e-3 * 0.01) - 1e-3 * (m / (1 - 0.9 ** t)) / (np.sqrt(v / (1 - 0.999 ** t)) + 1e-8)
    assert np.abs(th - ref).max() <= 5e-3 * 1e-3
    for b_out in (4, 8):
        co, so = O.repack(st.v_codes, st.v_scales, 16, b_out, n, block, O.LOG_TS)
        assert (so.view(np.uint32) == st.v_scales.view(np.uint32)).all()
        cb, sb = O.repack(co, so, b_out, 16, n, block, O.LOG_TS)
        c1, s1 = O.repack(cb, sb, 16, b_out, n, block, O.LOG_TS)
        assert (c1 == co).all() and (s1.view(np.uint32) == so.view(np.uint32)).all()

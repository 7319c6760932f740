"""Pins for the oracle's quantizers: worked examples, closed forms, invariants (CPU only)."""
import os

import numpy as np
import pytest

GOLD = os.path.join(os.path.dirname(__file__), "golden")
WIDTHS = (2, 3, 4, 8, 16)


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                yield [p.split() for p in line.split("|")]


# ---- worked examples ---------------------------------------------------------------------------
def test_worked_examples(O):
    n_seen = 0
    for head, xs, codes, decoded in _rows("quant_worked_examples.txt"):
        if head[0] == "ts":          # the two-scale lines are read by the pins of that variant
            continue
        mode = O.LINEAR if head[0] == "lin" else O.LOG
        bits, scale = int(head[1]), float(head[2])
        x = np.array([float(v) for v in xs], dtype=np.float32)
        c, s = O.quantize(x, bits, 128, mode)
        assert s[0] == np.float32(scale)
        got = O.unpack(c, x.size, bits)
        assert got.tolist() == [int(v) for v in codes], (head, got)
        xh = O.dequantize(c, s, x.size, bits, 128, mode)
        np.testing.assert_allclose(xh, np.array([float(v) for v in decoded]), rtol=1e-6, atol=0)
        n_seen += 1
    assert n_seen == 6


def test_pack_bytes_by_hand(O):
    seen = set()
    for head, hexbytes in _rows("pack_example.txt"):
        b = int(head[0])
        code = np.array([(5 * i + 3) % (1 << b) for i in range(16)], dtype=np.uint32)
        buf = O.pack(code, b)
        assert buf.tolist() == [int(h, 16) for h in hexbytes], b
        seen.add(b)
    assert seen == set(WIDTHS)


@pytest.mark.parametrize("bits", WIDTHS)
@pytest.mark.parametrize("n", [1, 7, 8, 9, 127, 128, 129, 1000])
def test_pack_roundtrip_all_values(O, bits, n):
    rng = np.random.default_rng(bits * 1000 + n)
    code = rng.integers(0, 1 << bits, size=n, dtype=np.uint32)
    code[: min(n, 2)] = [(1 << bits) - 1, 0][: min(n, 2)]
    buf = O.pack(code, bits)
    assert buf.size == ((n * bits + 7) // 8 + 15) // 16 * 16
    assert (O.unpack(buf, n, bits) == code).all()
    # independent bit-level check of the layout
    bitsarr = np.unpackbits(buf, bitorder="little")
    for i in (0, n // 2, n - 1):
        v = sum(int(bitsarr[i * bits + k]) << k for k in range(bits))
        assert v == code[i]
    assert bitsarr[n * bits:].sum() == 0   # padding is zero


# ---- lg / ex against the library functions ------------------------------------------------------
def test_lg_matches_log2(O):
    rng = np.random.default_rng(1)
    xs = np.concatenate([np.exp2(rng.uniform(-100, 100, 20000)), [1.0, 2.0, 0.5, 1.9999999, 1.0000001]])
    worst = 0.0
    for x in xs.astype(np.float32):
        lg = (O.lg_E(x) - 127) + O.lg_P(x)
        worst = max(worst, abs(lg - np.log2(np.float64(x))))
    assert worst <= 4e-6, worst
    assert O.lg_P(1.0) == 0.0 and O.lg_P(4.0) == 0.0 and O.lg_E(1.0) == 127


def test_ex_matches_exp2(O):
    rng = np.random.default_rng(2)
    worst = 0.0
    for e in np.concatenate([rng.uniform(-30, 0, 20000), np.arange(-30, 1), np.arange(-30, 0) + 0.5]).astype(np.float32):
        worst = max(worst, abs(O.ex2(e) / np.exp2(np.float64(e)) - 1))
    assert worst <= 4e-7, worst
    assert O.ex2(0.0) == 1.0
    for k in range(0, 31):
        assert O.ex2(-float(k)) == 2.0 ** -k    # whole octaves are exact


# ---- linear quantizer ---------------------------------------------------------------------------
def _heavy(rng, n, scale=1e-3):
    return (rng.standard_t(4, size=n) * scale).astype(np.float32)


@pytest.mark.parametrize("bits", WIDTHS)
@pytest.mark.parametrize("block", [128, 256])
def test_linear_half_step_and_max(O, bits, block):
    rng = np.random.default_rng(bits)
    n = block * 97 + 37
    x = _heavy(rng, n)
    c, s = O.quantize(x, bits, block, O.LINEAR)
    xh = O.dequantize(c, s, n, bits, block, O.LINEAR)
    qmax = (1 << (bits - 1)) - 1
    sx = np.repeat(s, block)[:n].astype(np.float64)
    step = sx / qmax
    bound = step * (0.5 + qmax * 2.0 ** -22) + np.abs(x) * 2.0 ** -23
    assert (np.abs(x.astype(np.float64) - xh) <= bound).all()
    # scale is the block absmax and the extreme element decodes to exactly +-scale
    pad = np.zeros(s.size * block, np.float32)
    pad[:n] = x
    blk = pad.reshape(-1, block)
    assert (np.abs(blk).max(1) == s).all()
    padh = np.zeros_like(pad)
    padh[:n] = xh
    j = np.abs(blk).argmax(1)
    rows = np.arange(s.size)
    assert (padh.reshape(-1, block)[rows, j] == blk[rows, j]).all()
    codes = O.unpack(c, n, bits)
    assert codes.min() >= 1 and codes.max() <= 2 * qmax + 1   # code 0 is never produced


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("bits", WIDTHS)
def test_idempotent_codes_and_scales(O, mode, bits):
    rng = np.random.default_rng(10 + bits)
    n = 128 * 300 + 5
    x = _heavy(rng, n)
    if mode == 1:
        x = x * x
    c, s = O.quantize(x, bits, 128, mode)
    xh = O.dequantize(c, s, n, bits, 128, mode)
    c2, s2 = O.quantize(xh, bits, 128, mode)
    assert (c == c2).all() and (s == s2).all()


def test_linear_bound_and_rms_monotone_in_bits(O):
    rng = np.random.default_rng(5)
    n = 128 * 500
    x = _heavy(rng, n)
    rms = []
    for b in WIDTHS:
        c, s = O.quantize(x, b, 128, O.LINEAR)
        xh = O.dequantize(c, s, n, b, 128, O.LINEAR)
        rms.append(float(np.sqrt(np.mean((x.astype(np.float64) - xh) ** 2))))
    assert all(a > b for a, b in zip(rms, rms[1:])), rms
    half_steps = [1.0 / (2 * ((1 << (b - 1)) - 1)) for b in WIDTHS]
    assert all(a > b for a, b in zip(half_steps, half_steps[1:]))


def test_zero_and_tiny_blocks(O):
    for bits in WIDTHS:
        x = np.zeros(256, np.float32)
        x[128:] = 1e-35   # below the tiny-scale rule (2^-100 ~ 7.9e-31)
        for mode in (0, 1):
            c, s = O.quantize(x, bits, 128, mode)
            assert (s == 0).all()
            codes = O.unpack(c, 256, bits)
            assert (codes == ((1 << (bits - 1)) if mode == 0 else 0)).all()
            assert (O.dequantize(c, s, 256, bits, 128, mode) == 0).all()


# ---- log quantizer ------------------------------------------------------------------------------
@pytest.mark.parametrize("bits", WIDTHS)
def test_log_error_floor_and_levels(O, bits):
    rng = np.random.default_rng(20 + bits)
    n = 128 * 211 + 19
    x = (_heavy(rng, n) ** 2).astype(np.float32)
    x[::97] = 0.0
    c, s = O.quantize(x, bits, 128, O.LOG)
    xh = O.dequantize(c, s, n, bits, 128, O.LOG).astype(np.float64)
    codes = O.unpack(c, n, bits)
    K = (1 << bits) - 1
    R = min(K, 30)
    sx = np.repeat(s, 128)[:n].astype(np.float64)
    floor = sx * 2.0 ** -R
    inr = x.astype(np.float64) >= floor
    err = np.abs(np.log2(xh[inr]) - np.log2(x[inr].astype(np.float64)))
    assert err.max() <= (R / K) / 2 * 1.05
    # below the floor: code 0 (or 1 within half a step of the floor), never an exact zero
    low = ~inr
    assert (codes[low] <= 1).all() and (xh[low] > 0).all()
    np.testing.assert_allclose(xh[codes == 0], floor[codes == 0], rtol=1e-6)
    # the block maximum is code K and decodes to exactly the scale
    assert (xh[codes == K] == sx[codes == K]).all()
    pad = np.zeros(s.size * 128, np.float32)
    pad[:n] = x
    assert (pad.reshape(-1, 128).max(1) == s).all()
    if bits <= 4:   # one octave per code: decoded values are the scale times a power of two
        assert (xh == sx * np.exp2(codes.astype(np.float64) - K)).all()


def test_log_nested_levels_and_rms(O):
    rng = np.random.default_rng(30)
    n = 128 * 400
    x = (_heavy(rng, n) ** 2).astype(np.float32)
    errs = {}
    for b in WIDTHS:
        c, s = O.quantize(x, b, 128, O.LOG)
        xh = O.dequantize(c, s, n, b, 128, O.LOG).astype(np.float64)
        errs[b] = np.abs(np.log2(xh) - np.log2(np.maximum(x.astype(np.float64), 1e-300)))
    # level sets are nested for 2 within 4 and 8 within 16, so the finer code is never worse
    # (up to the polynomial's few-1e-6 octaves)
    pos = x > 0
    assert (errs[4][pos] <= errs[2][pos] + 1e-5).all()
    assert (errs[16][pos] <= errs[8][pos] + 1e-5).all()
    rms = [float(np.sqrt(np.mean(errs[b][pos] ** 2))) for b in WIDTHS]
    assert all(a >= b for a, b in zip(rms, rms[1:])), rms


def test_log_monotone_codes(O):
    # a larger value never gets a smaller code
    for bits in WIDTHS:
        x = np.exp2(np.linspace(-35, 0, 128 * 40)).astype(np.float32)
        x = x.reshape(40, 128)
        x[:, -1] = 1.0
        c, s = O.quantize(x.ravel(), bits, 128, O.LOG)
        codes = O.unpack(c, x.size, bits).reshape(40, 128)[:, :-1].ravel().astype(np.int64)
        assert (np.diff(codes) >= 0).all()


# ---- repack -------------------------------------------------------------------------------------
@pytest.mark.parametrize("mode", [0, 1])
def test_repack_properties(O, mode):
    rng = np.random.default_rng(40 + mode)
    n = 128 * 50 + 77
    x = _heavy(rng, n)
    if mode == 1:
        x = x * x
    for b in WIDTHS:
        c, s = O.quantize(x, b, 128, mode)
        c_same, s_same = O.repack(c, s, b, b, n, 128, mode)
        assert (c_same == c).all() and (s_same == s).all()
        for b2 in WIDTHS:
            c2, s2 = O.repack(c, s, b, b2, n, 128, mode)
            assert (s2 == s).all()                       # scales survive a width change
            if b2 > b:                                   # widening and coming back is lossless
                c3, s3 = O.repack(c2, s2, b2, b, n, 128, mode)
                assert (c3 == c).all() and (s3 == s).all()
        # to 32 bits = plain decode; from raw fp32 = plain quantize
        raw, _ = O.repack(c, s, b, 32, n, 128, mode)
        assert (raw.view(np.float32)[:n] == O.dequantize(c, s, n, b, 128, mode)).all()
        xb = x.view(np.uint8).copy()
        cq, sq = O.repack(xb, np.zeros(0, np.float32), 32, b, n, 128, mode)
        assert (cq == c).all() and (sq == s).all()

"""Do the pins notice a broken oracle?

Each case below plants one plausible mistake (a dropped term, a wrong sign, a swapped coefficient, an
off-by-one, a transposed bit order) into a copy of the oracle's source, builds it, and runs the pin
suite against the broken build in a subprocess.  The suite must fail every time: a mutant that
survives is a hole in the pins."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "stq_oracle.cpp")
PIN_FILES = ["tests/test_oracle_quantizer.py", "tests/test_oracle_adamw.py", "tests/test_oracle_policy.py",
             "tests/test_oracle_quantizer_pl.py"]

# (name, text in the oracle, replacement)
MUTANTS = [
    ("betas swapped in the first moment", "m[i] = fmaf(fb1, m[i], c);", "m[i] = fmaf(fb2, m[i], c);"),
    ("second moment from g instead of g^2", "float w2 = w * g[i];", "float w2 = w;"),
    ("update added instead of subtracted", "* decay - lr * mt /", "* decay + lr * mt /"),
    ("decoupled decay dropped", "hp->decoupled_wd ? 1.0 - lr * (double)hp->weight_decay : 1.0", "1.0"),
    ("bias correction of v from beta1", "1.0 - std::pow(b2, (double)hp->step)", "1.0 - std::pow(b1, (double)hp->step)"),
    ("epsilon inside the square root", "(std::sqrt(vt) + eps)", "std::sqrt(vt + eps)"),
    ("update from the unquantized moments",
     "decode_state(m_codes_out, m_scales_out, n, bits_m_out, block, 0, m.data());", ""),
    ("linear code truncates instead of rounding", "double r = nearbyint((double)x[i] * (double)inv);",
     "double r = std::trunc((double)x[i] * (double)inv);"),
    ("linear scale without the absolute value", "float a = fabsf(x[i]); if (a > s) s = a;", "float a = x[i]; if (a > s) s = a;"),
    ("linear code offset by qmax instead of 2^(b-1)", "code[i] = (uint32_t)((int)r + half);", "code[i] = (uint32_t)((int)r + qmax);"),
    ("octave code off by one", "int q = K + (lg_E(y) - 127);", "int q = K + (lg_E(y) - 126);"),
    ("octave code floors instead of rounding to the nearest octave", "const float c = rs * kSqrt2;", "const float c = rs;"),
    ("log decode with the wrong step", "float e = rf * c_b;", "float e = rf * (1.0f / (float)K);"),
    ("log code ignores the exponent difference", "float d = de + dp;", "float d = dp;"),
    ("bitstream most-significant bit first",
     "v |= (uint32_t)((s[bit >> 3] >> (bit & 7)) & 1u) << k;", "v |= (uint32_t)((s[bit >> 3] >> (7 - (bit & 7))) & 1u) << k;",
     "uint8_t m = (uint8_t)(1u << (bit & 7));", "uint8_t m = (uint8_t)(1u << (7 - (bit & 7)));"),
    ("sum of |g| without the absolute value", "sa += fabs(gd);", "sa += gd;"),
    ("score without the annealing term", "std::log2(n[l] / (p->n_ema + p->eps_stat)) + std::log2(S) +",
     "std::log2(n[l] / (p->n_ema + p->eps_stat)) +"),
    ("score offset", "double sc = 7.2 +", "double sc = 7.0 +"),
    ("running averages updated after the scores", "p->r_ema = p->alpha * (sr / L) + (1 - p->alpha) * p->r_ema;", ""),
    ("variation factor from the signed mean", "double var = p->cv_of_signed ? mean_sq - mean * mean : mean_sq - mean_abs * mean_abs;",
     "double var = mean_sq - mean * mean;"),
    ("pl code floors instead of rounding", "int64_t j = (2 * dist * K + D) / (2 * D);", "int64_t j = (dist * K) / D;"),
    ("pl decode without the rounding term", "(j * pl_step(b) + ((int64_t)1 << (S - 1))) >> S", "(j * pl_step(b)) >> S"),
    ("zero-block rule missing for v", "if (s < kTinyScale) {\n    *scale = 0.0f;\n    for (uint64_t i = 0; i < n; ++i) code[i] = 0u;",
     "if (false) {\n    *scale = 0.0f;\n    for (uint64_t i = 0; i < n; ++i) code[i] = 0u;"),
    ("first moment's new term without 1 - beta1", "float c = omb1 * g[i];", "float c = g[i];"),
    ("1 - beta2 subtracted in single precision", "omb2 = (float)(1.0 - hp->beta2);", "omb2 = 1.0f - fb2;"),
    ("L2 term dropped", "float l2 = wd * theta[i]; g[i] = g[i] + l2;", "float l2 = wd * theta[i]; (void)l2;"),
    ("sum of squares from |g|", "sq += gd * gd;", "sq += fabs(gd);"),
    ("8/16-bit log code floors", "double r = nearbyint((double)d * (double)a_b);", "double r = std::floor((double)d * (double)a_b);"),
    ("2^e reduced by floor instead of nearest", "float i = nearbyintf(e);", "float i = floorf(e);"),
    ("skipped step is not skipped", "if (hp->found_inf) return 0;", "if (false) return 0;"),
    ("loss scale ignored", "grad_to_f32(grad, hp->grad_dtype, i) * hp->inv_grad_scale;", "grad_to_f32(grad, hp->grad_dtype, i);"),
    ("fp16 exponent bias off by one", "(uint32_t)(e + 112) << 23", "(uint32_t)(e + 111) << 23"),
    ("bf16 rounds half up", "(u + 0x7FFFu + ((u >> 16) & 1u)) >> 16", "(u + 0x8000u) >> 16"),
    ("zero-block threshold at the smallest normal", "const float kTinyScale = 0x1p-100f;", "const float kTinyScale = 0x1p-126f;"),
    ("scale of the neighbouring block", "float s = scales[i / block];", "float s = scales[(i + 1) / block];"),
    ("8-bit threshold moved", "sc < 12.0 ? 8", "sc < 13.0 ? 8"),
    ("annealing time constant inverted", "std::cosh((double)t / p->tau)", "std::cosh((double)t * p->tau)"),
    ("early decision steps end at t < 4", "(t % U == 0) || (t < 5)", "(t % U == 0) || (t < 4)"),
    ("running average weights swapped", "p->n_ema = p->alpha * (sn / L) + (1 - p->alpha) * p->n_ema;",
     "p->n_ema = (1 - p->alpha) * (sn / L) + p->alpha * p->n_ema;"),
    ("hierarchical factor from the mean instead of the mean square", "v[l] = mean_sq;", "v[l] = mean_abs;"),
]


# the two further readings of the logarithmic mode have their own pins (the 2^32-word enumerations are left
# out of the mutant runs: the closed-form threshold test covers the same ground in a fraction of the time)
VARIANT_PINS = ["tests/test_oracle_quantizer_variants.py", "tests/test_oracle_adamw.py", "-k", "not exact_enumeration"]
VARIANT_MUTANTS = [
    ("sr: scale nudge dropped, the maximum can fall below the top level", "const float c1 = rs * kOnePlus;", "const float c1 = rs;"),
    ("sr: the random word is ignored (round to nearest)", "int64_t j = ((n << (9 + g)) + (int64_t)U) >> 32;",
     "int64_t j = ((n << (9 + g)) + ((int64_t)1 << 31)) >> 32;"),
    ("sr: level spacing off by a factor of two", "int64_t j = ((n << (9 + g)) + (int64_t)U) >> 32;",
     "int64_t j = ((n << (8 + g)) + (int64_t)U) >> 32;"),
    ("sr: decode with the wrong level spacing", "(j << (23 - sr_lg_levels(b)))", "(j << (22 - sr_lg_levels(b)))"),
    ("sr: key ignores the tensor", "return mix32(tensor ^ h);", "return mix32(h);"),
    ("sr: words taken from the position in the block, not in the tensor", "sr_word(*key, e0 + j + i)", "sr_word(*key, i)"),
    ("sr: a range forgets where it starts in its tensor", "sr_word(*key, e0 + j + i)", "sr_word(*key, j + i)"),
    ("sr: a shift of the mixing function changed", "h ^= h >> 13;", "h ^= h >> 12;"),
    ("ts: minimum not raised to the floor", "if (lo < floor_level) lo = floor_level;", ""),
    ("ts: code 0 not the stored minimum", "if (code == 0u) return t.lo;", ""),
    ("ts: K + 1 steps instead of K", "const float inv = (float)K / t.W;", "const float inv = (float)(K + 1) / t.W;"),
    ("ts: both scales read from the first slot", "scales[2 * (i / block) + 1]", "scales[2 * (i / block)]"),
    ("ts: distance taken without the exponent difference", "float de = (float)(lg_E(x) - t.Ehi);\n  float dp = lg_P(x) - t.Phi;\n  return de + dp;",
     "float dp = lg_P(x) - t.Phi;\n  return dp;"),
]


def _build(tmp, idx, edits):
    import oracle
    src = open(SRC).read()
    for old, new in zip(edits[0::2], edits[1::2]):
        assert src.count(old) >= 1, f"mutant {idx}: the text to replace is not in the oracle: {old!r}"
        src = src.replace(old, new)
    cpp = os.path.join(tmp, f"mutant{idx}.cpp")
    so = os.path.join(tmp, f"mutant{idx}.so")
    with open(cpp, "w") as f:
        f.write(src)
    subprocess.check_call(["g++", *oracle.CXXFLAGS, "-w", "-o", so, cpp])
    return so


def _pins_fail(so, pins=None):
    env = dict(os.environ, STQ_ORACLE_LIB=so)
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", *(pins or PIN_FILES)],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    return r.returncode != 0, r.stdout[-400:]


def test_the_unbroken_oracle_passes_through_the_same_route(tmp_path):
    so = _build(str(tmp_path), "ok", ())
    failed, tail = _pins_fail(so)
    assert not failed, tail


def test_every_planted_mistake_is_caught(tmp_path):
    libs = [(m[0], _build(str(tmp_path), i, m[1:])) for i, m in enumerate(MUTANTS)]
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        results = list(ex.map(lambda nl: (nl[0], _pins_fail(nl[1])), libs))
    survivors = [name for name, (failed, _) in results if not failed]
    assert not survivors, "the pins do not notice: " + "; ".join(survivors)


def test_every_planted_mistake_in_the_variants_is_caught(tmp_path):
    ok = _build(str(tmp_path), "ok2", ())
    failed, tail = _pins_fail(ok, VARIANT_PINS)
    assert not failed, tail
    libs = [(m[0], _build(str(tmp_path), f"v{i}", m[1:])) for i, m in enumerate(VARIANT_MUTANTS)]
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        results = list(ex.map(lambda nl: (nl[0], _pins_fail(nl[1], VARIANT_PINS)), libs))
    survivors = [name for name, (failed, _) in results if not failed]
    assert not survivors, "the pins do not notice: " + "; ".join(survivors)

// CPU oracle for the mixed-bit quantized AdamW step (STQuant, Algorithm 1 and Sec. 3.3-3.5).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the hot path
// computes.  It is used by the tests, by the smoke check and by the timed CPU-baseline leg of the
// benchmark; the product path never calls it and shares no code, header or table with it.
//
// Everything is written element by element in the order the paper's Algorithm 1 states, with no
// blocking, fusion or reordering.  fp32 operations are single IEEE round-to-nearest-even
// operations (build with -ffp-contract=off, no fast-math); `fmaf` appears only where the
// quantizer definition says "fused".  Rounding-to-integer steps are taken on the exact product,
// which a double holds exactly for two fp32 factors.
//
// Parity status: the quantizer formulas are this build's reading of "linear symmetric" and
// "logarithmic" block-wise quantization (Sec. 3.5 gives no formula); they are pinned by the
// properties the tests check (half-step error bound, idempotence, monotone bound, exact block
// maximum, agreement with library AdamW at 32 and 16 bits).  The claim that ~5 bits preserve
// model quality needs the paper's training runs: parity unpinned for that claim.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

inline uint32_t f2u(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
inline float u2f(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

// A block whose maximum is below this is stored as an all-zero block (scale 0).
const float kTinyScale = 0x1p-100f;

// ---- widths ---------------------------------------------------------------------------------
inline bool width_ok(int b) { return b == 2 || b == 3 || b == 4 || b == 8 || b == 16 || b == 32; }
inline int qmax_of(int b) { return (1 << (b - 1)) - 1; }   // linear: largest |q|
inline int half_of(int b) { return 1 << (b - 1); }         // linear: offset of the stored code
inline int K_of(int b) { return (1 << b) - 1; }            // log: largest code
inline int R_of(int b) { int K = K_of(b); return K < 30 ? K : 30; }   // log: octaves covered

// ---- bitstream (LSB-first, little-endian; element i occupies bits [i*b, (i+1)*b)) ------------
inline uint32_t get_code(const uint8_t* s, uint64_t i, int b) {
  uint64_t bit = i * (uint64_t)b;
  uint32_t v = 0;
  for (int k = 0; k < b; ++k, ++bit) v |= (uint32_t)((s[bit >> 3] >> (bit & 7)) & 1u) << k;
  return v;
}
inline void put_code(uint8_t* s, uint64_t i, int b, uint32_t v) {
  uint64_t bit = i * (uint64_t)b;
  for (int k = 0; k < b; ++k, ++bit) {
    uint8_t m = (uint8_t)(1u << (bit & 7));
    if ((v >> k) & 1u) s[bit >> 3] |= m; else s[bit >> 3] &= (uint8_t)~m;
  }
}
inline uint64_t codes_bytes(uint64_t n, int b) {
  uint64_t by = (n * (uint64_t)b + 7) / 8;
  return (by + 15) / 16 * 16;
}

// ---- lg: split base-2 logarithm of a non-negative float -------------------------------------
// lg(x) = (E - 127) + P(t), E the biased exponent field, t = mantissa field * 2^-23 in [0,1),
// P(t) = t*(c1 + t*(c2 + ... + t*c6)) ~ log2(1+t), Horner with fused steps, final multiply rounded.
// (For zero/denormal inputs the fields are used literally; such values only occur in blocks that
// the tiny-scale rule zeroes or far below the coding floor.)
const float kP1 = 0x1.714b30p+0f, kP2 = -0x1.6fc360p-1f, kP3 = 0x1.d54a42p-2f,
            kP4 = -0x1.1e4792p-2f, kP5 = 0x1.f9c008p-4f, kP6 = -0x1.b19412p-6f;
inline int lg_E(float x) { return (int)(f2u(x) >> 23); }
inline float lg_P(float x) {
  float mant = u2f((f2u(x) & 0x007FFFFFu) | 0x3F800000u);
  float t = mant - 1.0f;
  float a = kP6;
  a = fmaf(a, t, kP5);
  a = fmaf(a, t, kP4);
  a = fmaf(a, t, kP3);
  a = fmaf(a, t, kP2);
  a = fmaf(a, t, kP1);
  return a * t;
}

// ---- ex: 2^e for e <= 0 -----------------------------------------------------------------------
// i = round-half-even(e), f = e - i in [-1/2, 1/2], p = 1 + f*(e0 + f*(e1 + ... + f*e4)) fused,
// ex = p * 2^i (exact scaling).  ex(0) == 1 exactly.
const float kE0 = 0x1.62e42ap-1f, kE1 = 0x1.ebf9bcp-3f, kE2 = 0x1.c6b74cp-5f,
            kE3 = 0x1.3cea84p-7f, kE4 = 0x1.5bbc6ap-10f;
inline float ex2(float e) {
  float i = nearbyintf(e);
  float f = e - i;
  float a = kE4;
  a = fmaf(a, f, kE3);
  a = fmaf(a, f, kE2);
  a = fmaf(a, f, kE1);
  a = fmaf(a, f, kE0);
  float p = fmaf(a, f, 1.0f);
  return ldexpf(p, (int)i);
}

// ---- linear symmetric block quantizer (first moment) ----------------------------------------
// scale s = max|x|; inv = fl(qmax * fl(1/s)); q = clamp(round-half-even(x * inv), -qmax, qmax);
// stored code q + 2^(b-1).
void quant_lin_block(const float* x, uint64_t n, int b, uint32_t* code, float* scale) {
  float s = 0.0f;
  for (uint64_t i = 0; i < n; ++i) { float a = fabsf(x[i]); if (a > s) s = a; }
  const int qmax = qmax_of(b), half = half_of(b);
  if (s < kTinyScale) {
    *scale = 0.0f;
    for (uint64_t i = 0; i < n; ++i) code[i] = (uint32_t)half;
    return;
  }
  *scale = s;
  float rs = 1.0f / s;
  float inv = (float)qmax * rs;
  for (uint64_t i = 0; i < n; ++i) {
    double r = nearbyint((double)x[i] * (double)inv);
    if (r > qmax) r = qmax;
    if (r < -qmax) r = -qmax;
    code[i] = (uint32_t)((int)r + half);
  }
}
inline float dequant_lin(uint32_t code, float s, int b) {
  float invq = 1.0f / (float)qmax_of(b);
  float q = (float)((int)code - half_of(b));
  float y = q * invq;
  return s * y;
}

// ---- logarithmic block quantizer (second moment, x >= 0) -------------------------------------
// scale s = max x; code K is the block maximum, each code step is R/K octaves, code 0 is the floor
// s*2^-R.
//  * b <= 4 (R = K, one octave per code): the code is the nearest octave below the maximum,
//    q = clamp(K + floor(log2(x/s) + 1/2), 0, K), taken as the exponent of y = fl(x * c) with
//    c = fl(fl(1/s) * sqrt2): floor(log2(x*sqrt2/s)) is that exponent.
//  * b = 8, 16: d = log-distance to the maximum in octaves from the split logarithm,
//    q = clamp(K + round-half-even(d*K/R), 0, K).
//
// Variant "pl" (mode 2; an alternative reading of "logarithmic", integer-only at widths 8 and 16):
// the logarithm is replaced by the piecewise-linear one that the fp32 bit pattern itself is,
// pl(x) = bits(x) * 2^-23 - 127 (equal to log2 at powers of two, linear in the mantissa between them).
// With D = R * 2^23 (R octaves in units of the bit pattern), all in exact integers:
//  * n = min(bits(s) - bits(x), D), the distance below the block maximum;
//    j = floor(n*K/D + 1/2) code steps below the maximum; q = K - j.
//  * decode: j = K - q; n' = floor(j*B/2^S + 1/2) with B = round(D * 2^S / K) and S = 12 (8 bits),
//    20 (16 bits), so that j*B fits 64 bits with B below 2^32; bits(x^) = max(bits(s) - n', 0).
//    n' = k * 2^23 exactly whenever j is a whole number k of octaves.
//  * widths <= 4 are the octave code above in both variants.
const float kSqrt2 = 0x1.6a09e6p+0f;
inline int pl_shift(int b) { return b == 8 ? 12 : 20; }
inline int64_t pl_octaves(int b) { return (int64_t)R_of(b) << 23; }                    // D
inline int64_t pl_step(int b) {                                                        // B
  const int64_t K = K_of(b), D = pl_octaves(b);
  return (2 * (D << pl_shift(b)) + K) / (2 * K);
}
// Variant "sr" (mode 3; the third reading of "logarithmic": the piecewise-linear logarithm of x/s with
// STOCHASTIC rounding, so that the stored second moment is an unbiased estimate of the one computed).
// The level grid has a whole number of levels per octave, L = 1, 1, 1, 8, 2048 at widths 2, 3, 4, 8, 16
// (g = log2 L = 0, 0, 0, 3, 11), so every power of two below the maximum is a level and the code covers
// K / L octaves (3, 7, 15, 31.875, 32.0).
//  * c1 = fl(fl(1/s) * (1 + 2^-21)); y = fl(x * c1): the block maximum lands at or just above 1, never below.
//  * n = clamp(bits(1.0) - bits(y), 0, K << (23 - g)): distance below the maximum in units of the bit
//    pattern, i.e. -2^23 times the piecewise-linear log2 of y.
//  * j = min(((n << (9 + g)) + U) >> 32, K), U the 32-bit random word of the element: j = floor(n * L / 2^23
//    + U / 2^32), the lower neighbour with probability 1 - frac and the upper one with probability frac.
//    Code q = K - j.
//  * decode: y^ = the float with bits(1.0) - (j << (23 - g)); x^ = fl(s * y^).
// Between two neighbouring levels there is no power of two, so the bit pattern is linear in y there and
// E[y^] = y EXACTLY, at every width (tests: exact enumeration over all 2^32 words, in rationals).
// Re-quantizing a decoded state is not the identity under random words (a level re-rounds to itself only
// when its y lands exactly on it): idempotence is given up for unbiasedness.
//
// The random word is a counter-based generator, keyed on (seed, step, tensor, element) and specified to
// the bit: mix32(h): h ^= h >> 16; h *= 0x85EBCA6B; h ^= h >> 13; h *= 0xC2B2AE35; h ^= h >> 16 (every
// step is invertible, so mix32 is a bijection of the 32-bit words);
// h = mix32(seed_lo ^ mix32(seed_hi ^ mix32(step_lo ^ mix32(step_hi ^ 0x9E3779B9)))) (one word per step);
// key = mix32(tensor ^ h); U(element e) = mix32(e_lo ^ mix32(key + e_hi)).  For a fixed key, e_lo -> U is a bijection: over any
// 2^32 consecutive elements every word occurs exactly once.
const float kOnePlus = 0x1.000008p+0f;      // 1 + 2^-21
inline uint32_t mix32(uint32_t h) {
  h ^= h >> 16; h *= 0x85EBCA6Bu; h ^= h >> 13; h *= 0xC2B2AE35u; h ^= h >> 16;
  return h;
}
inline uint32_t sr_key(uint64_t seed, uint64_t step, uint32_t tensor) {
  uint32_t h = mix32((uint32_t)(step >> 32) ^ 0x9E3779B9u);
  h = mix32((uint32_t)step ^ h);
  h = mix32((uint32_t)(seed >> 32) ^ h);
  h = mix32((uint32_t)seed ^ h);
  return mix32(tensor ^ h);
}
inline uint32_t sr_word(uint32_t key, uint64_t e) {
  return mix32((uint32_t)e ^ mix32(key + (uint32_t)(e >> 32)));
}
inline int sr_lg_levels(int b) { return b == 8 ? 3 : b == 16 ? 11 : 0; }      // g
inline uint32_t sr_code(float x, float s, int b, uint32_t U) {
  const int64_t K = K_of(b);
  const int g = sr_lg_levels(b);
  const float rs = 1.0f / s;
  const float c1 = rs * kOnePlus;
  const float y = x * c1;
  int64_t n = (int64_t)0x3F800000 - (int64_t)f2u(y);
  if (n < 0) n = 0;
  if (n > (K << (23 - g))) n = K << (23 - g);
  int64_t j = ((n << (9 + g)) + (int64_t)U) >> 32;
  if (j > K) j = K;
  return (uint32_t)(K - j);
}
inline float sr_level(uint32_t code, int b) {      // y^ of a code
  const int64_t j = (int64_t)K_of(b) - (int64_t)code;
  return u2f((uint32_t)((int64_t)0x3F800000 - (j << (23 - sr_lg_levels(b)))));
}

// Variant "ts" (mode 4; two scales per block): the codes are spread evenly, in the logarithm, between the
// block's own minimum and maximum instead of over a fixed number of octaves below the maximum.
//  * stored scales (two per block): hi = max x, lo = max(min x, fl(hi * 2^-30)) (at most 30 octaves; a
//    zero or denormal element is coded at the floor, never as zero).
//  * d(x) = fl( float(E_x - E_hi) + fl(P(x) - P(hi)) ), the split logarithm of x/hi as in the main code;
//    W = min(-d(lo), 30); inv = fl(K / W); q = clamp(K + round-half-even(d(x) * inv), 0, K) on the exact
//    product.  W = 0 (all elements equal): every code is K.
//  * decode: code 0 is lo exactly; otherwise x^ = fl(hi * ex(fl(float(q - K) * fl(W / K)))), so code K is
//    hi exactly.  |log2(x^/x)| <= W/(2K) for lo <= x <= hi (plus the ~4e-6 octaves of the polynomials).
struct TsBlock { float hi, lo, W; int Ehi; float Phi; };
inline float ts_dist(const TsBlock& t, float x) {
  float de = (float)(lg_E(x) - t.Ehi);
  float dp = lg_P(x) - t.Phi;
  return de + dp;
}
inline TsBlock ts_block(float hi, float lo) {
  TsBlock t;
  t.hi = hi; t.lo = lo; t.Ehi = lg_E(hi); t.Phi = lg_P(hi);
  float W = -ts_dist(t, lo);
  if (W > 30.0f) W = 30.0f;
  if (!(W > 0.0f)) W = 0.0f;
  t.W = W;
  return t;
}
void quant_ts_block(const float* x, uint64_t n, int b, uint32_t* code, float* scale2) {
  float hi = 0.0f;
  for (uint64_t i = 0; i < n; ++i) if (x[i] > hi) hi = x[i];
  if (hi < kTinyScale) {
    scale2[0] = 0.0f; scale2[1] = 0.0f;
    for (uint64_t i = 0; i < n; ++i) code[i] = 0u;
    return;
  }
  float lo = hi;
  for (uint64_t i = 0; i < n; ++i) if (x[i] < lo) lo = x[i];
  const float floor_level = hi * 0x1p-30f;
  if (lo < floor_level) lo = floor_level;
  scale2[0] = hi; scale2[1] = lo;
  const int K = K_of(b);
  const TsBlock t = ts_block(hi, lo);
  if (t.W == 0.0f) { for (uint64_t i = 0; i < n; ++i) code[i] = (uint32_t)K; return; }
  const float inv = (float)K / t.W;
  for (uint64_t i = 0; i < n; ++i) {
    float d = ts_dist(t, x[i]);
    double r = nearbyint((double)d * (double)inv);
    double q = (double)K + r;
    if (q < 0) q = 0;
    if (q > K) q = K;
    code[i] = (uint32_t)q;
  }
}
inline float dequant_ts(uint32_t code, const TsBlock& t, int b) {
  if (t.hi == 0.0f) return 0.0f;
  if (code == 0u) return t.lo;
  const int K = K_of(b);
  float step = t.W / (float)K;
  float e = (float)((int)code - K) * step;
  float y = ex2(e);
  return t.hi * y;
}

void quant_log_block(const float* x, uint64_t n, int b, uint32_t* code, float* scale, bool pl) {
  float s = 0.0f;
  for (uint64_t i = 0; i < n; ++i) if (x[i] > s) s = x[i];
  if (s < kTinyScale) {
    *scale = 0.0f;
    for (uint64_t i = 0; i < n; ++i) code[i] = 0u;
    return;
  }
  *scale = s;
  const int K = K_of(b), R = R_of(b);
  if (b <= 4) {
    const float rs = 1.0f / s;
    const float c = rs * kSqrt2;
    for (uint64_t i = 0; i < n; ++i) {
      float y = x[i] * c;
      int q = K + (lg_E(y) - 127);
      if (q < 0) q = 0;
      if (q > K) q = K;
      code[i] = (uint32_t)q;
    }
    return;
  }
  const float a_b = (float)K / (float)R;          // exact: 8.5, 2184.5
  if (pl) {
    const int64_t D = pl_octaves(b);
    for (uint64_t i = 0; i < n; ++i) {
      int64_t dist = (int64_t)f2u(s) - (int64_t)f2u(x[i]);
      if (dist > D) dist = D;
      int64_t j = (2 * dist * K + D) / (2 * D);   // floor(dist*K/D + 1/2)
      code[i] = (uint32_t)(K - j);
    }
    return;
  }
  const int Es = lg_E(s);
  const float Ps = lg_P(s);
  for (uint64_t i = 0; i < n; ++i) {
    float de = (float)(lg_E(x[i]) - Es);
    float dp = lg_P(x[i]) - Ps;
    float d = de + dp;
    double r = nearbyint((double)d * (double)a_b);
    double q = (double)K + r;
    if (q < 0) q = 0;
    if (q > K) q = K;
    code[i] = (uint32_t)q;
  }
}
inline float dequant_log(uint32_t code, float s, int b, bool pl) {
  const int K = K_of(b), R = R_of(b);
  const float c_b = (float)R / (float)K;
  float rf = (float)((int)code - K);
  if (pl && b > 4) {
    const int64_t j = (int64_t)K - (int64_t)code;
    const int S = pl_shift(b);
    const int64_t below = (j * pl_step(b) + ((int64_t)1 << (S - 1))) >> S;
    int64_t xb = (int64_t)f2u(s) - below;
    if (xb < 0) xb = 0;
    return u2f((uint32_t)xb);
  }
  float e = rf * c_b;
  float y = ex2(e);
  return s * y;
}

// ---- state (de)coding over a whole range ------------------------------------------------------
// mode 0 = linear (m), 1 = log (v), 2 = log with the piecewise-linear logarithm (v, variant "pl").
// Width 32 stores raw fp32 and no scales.
// mode 0 = linear (m), 1 = log (v), 2 = log with the piecewise-linear logarithm (v, variant "pl"),
// 3 = variant "sr" (stochastic rounding; `key` selects the random words), 4 = variant "ts" (two scales per
// block: scales[2k] = hi, scales[2k+1] = lo).  Width 32 stores raw fp32 and no scales.
inline uint64_t scales_per_block(int mode) { return mode == 4 ? 2 : 1; }
void decode_state(const uint8_t* codes, const float* scales, uint64_t n, int b, uint32_t block,
                  int mode, float* out) {
  if (b == 32) { std::memcpy(out, codes, n * 4); return; }
  TsBlock ts{};
  for (uint64_t i = 0; i < n; ++i) {
    uint32_t c = get_code(codes, i, b);
    if (mode == 4) {
      if (i % block == 0) ts = ts_block(scales[2 * (i / block)], scales[2 * (i / block) + 1]);
      out[i] = dequant_ts(c, ts, b);
      continue;
    }
    float s = scales[i / block];
    if (mode == 0) out[i] = dequant_lin(c, s, b);
    else if (mode == 3) { float lv = sr_level(c, b); out[i] = s * lv; }
    else out[i] = dequant_log(c, s, b, mode == 2);
  }
}
// key (variant "sr"): selects the random words, which belong to the elements' positions e0 + i in their
// tensor; without a key (a re-pack has no step to draw from) every word is 2^31, i.e. rounding to nearest.
void encode_state(const float* x, uint64_t n, int b, uint32_t block, int mode, uint8_t* codes,
                  float* scales, const uint32_t* key = nullptr, uint64_t e0 = 0) {
  if (b == 32) { std::memcpy(codes, x, n * 4); return; }
  std::memset(codes, 0, codes_bytes(n, b));
  std::vector<uint32_t> tmp(block);
  for (uint64_t j = 0, k = 0; j < n; j += block, ++k) {
    uint64_t len = n - j < block ? n - j : block;
    if (mode == 0) quant_lin_block(x + j, len, b, tmp.data(), scales + k);
    else if (mode == 4) quant_ts_block(x + j, len, b, tmp.data(), scales + 2 * k);
    else if (mode == 3) {
      float s = 0.0f;
      for (uint64_t i = 0; i < len; ++i) if (x[j + i] > s) s = x[j + i];
      if (s < kTinyScale) { scales[k] = 0.0f; for (uint64_t i = 0; i < len; ++i) tmp[i] = 0u; }
      else {
        scales[k] = s;
        for (uint64_t i = 0; i < len; ++i)
          tmp[i] = sr_code(x[j + i], s, b, key ? sr_word(*key, e0 + j + i) : 0x80000000u);
      }
    }
    else quant_log_block(x + j, len, b, tmp.data(), scales + k, mode == 2);
    for (uint64_t i = 0; i < len; ++i) put_code(codes, j + i, b, tmp[i]);
  }
}

inline float bf16_to_f32(uint16_t h) { return u2f((uint32_t)h << 16); }

// IEEE binary16 -> binary32 (exact).
inline float f16_to_f32(uint16_t h) {
  const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  const int e = (h >> 10) & 0x1F;
  const uint32_t m = h & 0x3FFu;
  if (e == 0) {                       // zero or subnormal: m * 2^-24
    const float v = (float)m * 0x1p-24f;
    return u2f(f2u(v) | sign);
  }
  if (e == 31) return u2f(sign | 0x7F800000u | (m << 13));
  return u2f(sign | ((uint32_t)(e + 112) << 23) | (m << 13));
}

// binary32 -> bfloat16 / binary16, round to nearest even (finite inputs).
inline uint16_t f32_to_bf16(float x) {
  const uint32_t u = f2u(x);
  return (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}
inline uint16_t f32_to_f16(float x) {
  const uint32_t u = f2u(x);
  const uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
  const float a = std::fabs(x);
  if (a >= 65520.0f) return sign | 0x7C00u;                 // rounds to infinity
  if (a < 0x1p-14f) {                                        // subnormal half: multiples of 2^-24
    const double q = std::nearbyint((double)a * 0x1p24);     // exact scaling, ties to even
    return sign | (uint16_t)q;                               // 1024 is the smallest normal: carries over correctly
  }
  const uint32_t au = f2u(a);
  const uint32_t rounded = au + 0xFFFu + ((au >> 13) & 1u);  // 13 mantissa bits dropped
  return sign | (uint16_t)(((rounded >> 13) - (112u << 10)) & 0x7FFFu);
}

inline float grad_to_f32(const void* grad, int dtype, uint64_t i) {
  if (dtype == 1) return bf16_to_f32(((const uint16_t*)grad)[i]);
  if (dtype == 2) return f16_to_f32(((const uint16_t*)grad)[i]);
  return ((const float*)grad)[i];
}

}  // namespace

extern "C" {

struct orc_hparams {
  double lr, beta1, beta2, eps, weight_decay;
  int64_t step;        // t >= 1, the step being taken
  int decoupled_wd;    // 1 = AdamW (Algorithm 1); 0 = L2 term added to the gradient
  int grad_dtype;      // 0 = fp32, 1 = bf16, 2 = fp16
  float inv_grad_scale;  // loss-scaled training: every gradient is multiplied by this first (1 = off)
  int found_inf;         // non-zero: a non-finite gradient was found, the step is skipped
  int v_mode;            // quantizer of the second moment: 1 = log, 2 = "pl", 3 = "sr", 4 = "ts"
  uint64_t sr_seed;      // variant "sr": the caller's seed ...
  uint32_t tensor_index; // ... and the index of this tensor in the caller's list (the step is `step`);
  uint64_t elem_offset;  // index of the range's first element inside its tensor (the random words are per element)
};

uint64_t orc_codes_bytes(uint64_t n, int bits) { return codes_bytes(n, bits); }
uint64_t orc_num_blocks(uint64_t n, uint32_t block) { return (n + block - 1) / block; }
uint64_t orc_num_scales(uint64_t n, uint32_t block, int mode) { return (n + block - 1) / block * scales_per_block(mode); }

// Test hooks of variant "sr": the generator and the rounding of one element given its random word.
uint32_t orc_mix32(uint32_t h) { return mix32(h); }
uint32_t orc_sr_key(uint64_t seed, uint64_t step, uint32_t tensor) { return sr_key(seed, step, tensor); }
uint32_t orc_sr_word(uint32_t key, uint64_t e) { return sr_word(key, e); }
uint32_t orc_sr_code(float x, float s, int bits, uint32_t U) { return sr_code(x, s, bits, U); }
float orc_sr_level(uint32_t code, int bits) { return sr_level(code, bits); }
// Exact enumeration: over ALL 2^32 random words, how often each code occurs for the element x of a block
// with maximum s (at most two neighbouring codes occur).  counts[0] goes with codes[0] (the smaller code).
void orc_sr_enumerate(float x, float s, int bits, uint32_t codes[2], uint64_t counts[2]) {
  codes[0] = sr_code(x, s, bits, 0xFFFFFFFFu);      // largest word: the lower level (larger j, smaller code)
  codes[1] = sr_code(x, s, bits, 0u);
  counts[0] = counts[1] = 0;
  for (uint64_t U = 0; U < ((uint64_t)1 << 32); ++U) {
    uint32_t c = sr_code(x, s, bits, (uint32_t)U);
    if (c == codes[1]) ++counts[1]; else if (c == codes[0]) ++counts[0]; else { counts[0] = counts[1] = ~(uint64_t)0; return; }
  }
}

float orc_lg_P(float x) { return lg_P(x); }
int orc_lg_E(float x) { return lg_E(x); }
float orc_ex2(float e) { return ex2(e); }

void orc_pack(const uint32_t* code, uint64_t n, int bits, uint8_t* out) {
  std::memset(out, 0, codes_bytes(n, bits));
  for (uint64_t i = 0; i < n; ++i) put_code(out, i, bits, code[i]);
}
void orc_unpack(const uint8_t* in, uint64_t n, int bits, uint32_t* code) {
  for (uint64_t i = 0; i < n; ++i) code[i] = get_code(in, i, bits);
}

// Quantize / dequantize a whole tensor state.  mode 0 = linear (m), 1 = log (v), 2 = log "pl" (v).
int orc_quantize(const float* x, uint64_t n, int bits, uint32_t block, int mode, uint8_t* codes,
                 float* scales) {
  if (!width_ok(bits) || block == 0) return -1;
  encode_state(x, n, bits, block, mode, codes, scales);
  return 0;
}
// The same with the key of variant "sr" (mode 3) given.
int orc_quantize_keyed(const float* x, uint64_t n, int bits, uint32_t block, int mode, uint32_t key, uint8_t* codes,
                       float* scales) {
  if (!width_ok(bits) || block == 0) return -1;
  encode_state(x, n, bits, block, mode, codes, scales, &key);
  return 0;
}
int orc_dequantize(const uint8_t* codes, const float* scales, uint64_t n, int bits, uint32_t block,
                   int mode, float* out) {
  if (!width_ok(bits) || block == 0) return -1;
  decode_state(codes, scales, n, bits, block, mode, out);
  return 0;
}

// Initial state (Algorithm 1, initialisation): m = v = 0 at the given widths.
int orc_init_state(uint64_t n, uint32_t block, int bits_m, int bits_v, uint8_t* m_codes,
                   float* m_scales, uint8_t* v_codes, float* v_scales) {
  std::vector<float> z(n, 0.0f);
  if (orc_quantize(z.data(), n, bits_m, block, 0, m_codes, m_scales)) return -1;
  if (orc_quantize(z.data(), n, bits_v, block, 1, v_codes, v_scales)) return -1;
  return 0;
}

// Per-layer gradient sums for the factor selection (Eq. 2, 3, 8): sum g, sum |g|, sum g^2, count.
void orc_grad_stats(const void* grad, int grad_dtype, uint64_t n, double out[4]) {
  double sg = 0, sa = 0, sq = 0;
  for (uint64_t i = 0; i < n; ++i) {
    float g = grad_to_f32(grad, grad_dtype, i);
    double gd = (double)g;
    sg += gd; sa += fabs(gd); sq += gd * gd;
  }
  out[0] = sg; out[1] = sa; out[2] = sq; out[3] = (double)n;
}

// One step of Algorithm 1's inner loop for one tensor (or any range that starts on a block
// boundary).  Stored states come in at (bits_m_in, bits_v_in) and leave at (bits_m_out,
// bits_v_out).  theta is updated in place.  stats, if non-null, receives the sums above.
int orc_step(float* theta, const void* grad, uint64_t n, uint32_t block,
             const uint8_t* m_codes_in, const float* m_scales_in, int bits_m_in,
             const uint8_t* v_codes_in, const float* v_scales_in, int bits_v_in,
             uint8_t* m_codes_out, float* m_scales_out, int bits_m_out,
             uint8_t* v_codes_out, float* v_scales_out, int bits_v_out,
             const orc_hparams* hp, double* stats) {
  if (!width_ok(bits_m_in) || !width_ok(bits_v_in) || !width_ok(bits_m_out) || !width_ok(bits_v_out))
    return -1;
  if (block == 0 || hp->step < 1) return -1;
  if (hp->v_mode < 1 || hp->v_mode > 4) return -1;
  if (hp->v_mode == 3 && hp->elem_offset % block != 0) return -1;
  const int vmode = hp->v_mode;
  if (hp->found_inf) return 0;          // skipped step: nothing is touched
  std::vector<float> m(n), v(n), g(n);

  // stored m_{t-1}, v_{t-1}
  decode_state(m_codes_in, m_scales_in, n, bits_m_in, block, 0, m.data());
  decode_state(v_codes_in, v_scales_in, n, bits_v_in, block, vmode, v.data());

  // gradient as fp32 (bf16 and fp16 widen exactly), brought back from the loss scale
  for (uint64_t i = 0; i < n; ++i) g[i] = grad_to_f32(grad, hp->grad_dtype, i) * hp->inv_grad_scale;
  if (stats) orc_grad_stats(g.data(), 0, n, stats);
  if (!hp->decoupled_wd) {
    const float wd = (float)hp->weight_decay;
    for (uint64_t i = 0; i < n; ++i) { float l2 = wd * theta[i]; g[i] = g[i] + l2; }
  }

  // moments: m_t = fma(b1, m, fl(c1*g)) ; v_t = fma(b2, v, fl(fl(c2*g)*g)) in fp32: the new term is
  // rounded, the decayed state is added with one fused rounding
  // (the four coefficients are the fp32 roundings of beta and of 1-beta taken in double)
  const float fb1 = (float)hp->beta1, fb2 = (float)hp->beta2;
  const float omb1 = (float)(1.0 - hp->beta1), omb2 = (float)(1.0 - hp->beta2);
  for (uint64_t i = 0; i < n; ++i) {
    float c = omb1 * g[i];
    m[i] = fmaf(fb1, m[i], c);
    float w = omb2 * g[i];
    float w2 = w * g[i];
    v[i] = fmaf(fb2, v[i], w2);
  }

  // Quantize(m_t, linear), Quantize(v_t, log) at the widths assigned for this step
  encode_state(m.data(), n, bits_m_out, block, 0, m_codes_out, m_scales_out);
  if (vmode == 3) {
    // the random words are those of the elements' positions in their tensor: a range is coded as the
    // elements [elem_offset, elem_offset + n) of the tensor it belongs to
    const uint32_t key = sr_key(hp->sr_seed, (uint64_t)hp->step, hp->tensor_index);
    encode_state(v.data(), n, bits_v_out, block, vmode, v_codes_out, v_scales_out, &key, hp->elem_offset);
  } else {
    encode_state(v.data(), n, bits_v_out, block, vmode, v_codes_out, v_scales_out);
  }

  // the update consumes the quantized states
  decode_state(m_codes_out, m_scales_out, n, bits_m_out, block, 0, m.data());
  decode_state(v_codes_out, v_scales_out, n, bits_v_out, block, vmode, v.data());

  const double b1 = hp->beta1, b2 = hp->beta2, lr = hp->lr, eps = hp->eps;
  const double bc1 = 1.0 - std::pow(b1, (double)hp->step);
  const double bc2 = 1.0 - std::pow(b2, (double)hp->step);
  const double decay = hp->decoupled_wd ? 1.0 - lr * (double)hp->weight_decay : 1.0;
  for (uint64_t i = 0; i < n; ++i) {
    double mt = (double)m[i] / bc1;
    double vt = (double)v[i] / bc2;
    double th = (double)theta[i] * decay - lr * mt / (std::sqrt(vt) + eps);
    theta[i] = (float)th;
  }
  return 0;
}

// Low-precision working copy of the parameters: nearest-even rounding to bf16 (1) or fp16 (2).
void orc_round_lp(const float* x, uint64_t n, int lp_dtype, uint16_t* out) {
  for (uint64_t i = 0; i < n; ++i) out[i] = lp_dtype == 1 ? f32_to_bf16(x[i]) : f32_to_f16(x[i]);
}
void orc_widen_f16(const uint16_t* x, uint64_t n, float* out) {
  for (uint64_t i = 0; i < n; ++i) out[i] = f16_to_f32(x[i]);
}

// Width transition: codes' = Q_{b'}(D_b(codes)), block scales recomputed from the decoded values
// (they come out unchanged whenever the source was itself quantized).
int orc_repack(const uint8_t* codes_in, const float* scales_in, int bits_in, uint8_t* codes_out,
               float* scales_out, int bits_out, uint64_t n, uint32_t block, int mode) {
  if (!width_ok(bits_in) || !width_ok(bits_out) || block == 0) return -1;
  std::vector<float> x(n);
  decode_state(codes_in, scales_in, n, bits_in, block, mode, x.data());
  encode_state(x.data(), n, bits_out, block, mode, codes_out, scales_out);
  return 0;
}

// ---- transition decision (Algorithm 1, decision branch; Sec. 3.3-3.4) -------------------------
struct orc_policy {
  double n_ema, r_ema, v_ema;   // global running statistics, start at 0
  double alpha, tau, eps_stat;
  int cv_of_signed;             // 0: sigma(|g|)/mu(|g|) (Eq. 3); 1: sigma(g)/E|g| (Algorithm 1)
};

int orc_is_decision_step(int64_t t, int64_t U) { return (t % U == 0) || (t < 5); }

// stats: L rows of {sum g, sum |g|, sum g^2, count}.  Writes bits[l] in {4,8,16,32} and, if
// non-null, score[l].  Updates the three running averages first, as Algorithm 1 orders it.
void orc_decide(orc_policy* p, const double* stats, int L, int64_t t, uint8_t* bits, double* score) {
  std::vector<double> n(L), r(L), v(L);
  double sn = 0, sr = 0, sv = 0;
  for (int l = 0; l < L; ++l) {
    const double* s = stats + 4 * l;
    double N = s[3];
    double mean_sq = s[2] / N;
    double mean_abs = s[1] / N;
    double mean = s[0] / N;
    n[l] = std::sqrt(mean_sq);
    v[l] = mean_sq;
    double var = p->cv_of_signed ? mean_sq - mean * mean : mean_sq - mean_abs * mean_abs;
    if (var < 0) var = 0;
    r[l] = std::sqrt(var) / (mean_abs + p->eps_stat);
    sn += n[l]; sr += r[l]; sv += v[l];
  }
  p->n_ema = p->alpha * (sn / L) + (1 - p->alpha) * p->n_ema;
  p->r_ema = p->alpha * (sr / L) + (1 - p->alpha) * p->r_ema;
  p->v_ema = p->alpha * (sv / L) + (1 - p->alpha) * p->v_ema;
  const double S = 1.0 + 1.0 / std::cosh((double)t / p->tau);
  for (int l = 0; l < L; ++l) {
    double sc = 7.2 + std::log2(r[l] / (p->r_ema + p->eps_stat)) +
                std::log2(n[l] / (p->n_ema + p->eps_stat)) + std::log2(S) +
                std::log2(v[l] / (p->v_ema + p->eps_stat));
    if (score) score[l] = sc;
    bits[l] = sc < 6.8 ? 4 : sc < 12.0 ? 8 : sc < 24.0 ? 16 : 32;
  }
}

}  // extern "C"

// Kernels of the mixed-bit quantized AdamW step for sm_100a.
//
// Generic path (ragged tails, 32-bit states, width changes, init, repack, statistics alone); the
// main step kernel is in stq_step_fast.cuh.
//
// Work decomposition: the concatenated tensor list is cut into tiles of kTile elements that never
// cross a tensor; persistent CTAs of 8 warps stride over the tile list.  Inside a tile a warp owns
// kRowsPerWarp consecutive rows of 128 elements and lane l of a row holds elements 4l..4l+3, so parameters
// and fp32 gradients move as 128-bit accesses (512 contiguous bytes per warp), bf16 gradients as
// 64-bit ones, and a lane's four codes are one 8/16/32/64-bit access at widths 2/4/8/16 (3-bit
// rows are 48 bytes: 12 lanes move one word each and the 12-bit lane fields are exchanged with
// shuffles).  A quantization block (128/256) is 1/2 whole rows of one warp, so the block
// maximum is a lane-local max of 4 followed by one warp REDUX on the (non-negative) bit patterns.
//
// Arithmetic that decides codes is written with the *_rn intrinsics, which are never contracted,
// and the file is compiled with -fmad=false; fused operations appear only where the quantizer is
// defined with them.  Round-half-even to integer is done by adding 1.5*2^23 (one FFMA on the exact
// product), and the integer sits in the low mantissa bits of the result, which is also how the
// codes are packed: sum_k bits_k << (k*b) minus a per-width constant.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "stq_internal.h"

namespace stq {
namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23: ulp 1, even
constexpr uint32_t kMagicBits = 0x4B400000u;   // its bit pattern (low 22 bits clear)
constexpr float kTwo23 = 8388608.0f;
constexpr uint32_t kTwo23Bits = 0x4B000000u;
constexpr float kTiny = 0x1p-100f;                //: smaller block maxima store a zero block
constexpr int kZeroBlockExp = 1 << 20;            // exponent stand-in that floors every log code
constexpr float kSqrt2 = 0x1.6a09e6p+0f;

// P(t) ~ log2(1+t) = t*(c1 + t*(c2 + ... + t*c6)), t in [0,1)
constexpr float kP1 = 0x1.714b30p+0f, kP2 = -0x1.6fc360p-1f, kP3 = 0x1.d54a42p-2f,
                kP4 = -0x1.1e4792p-2f, kP5 = 0x1.f9c008p-4f, kP6 = -0x1.b19412p-6f;
// 2^f ~ 1 + f*(e0 + f*(e1 + ... + f*e4)), |f| <= 1/2
constexpr float kE0 = 0x1.62e42ap-1f, kE1 = 0x1.ebf9bcp-3f, kE2 = 0x1.c6b74cp-5f,
                kE3 = 0x1.3cea84p-7f, kE4 = 0x1.5bbc6ap-10f;

__device__ __forceinline__ float lg_poly(uint32_t bits) {
  const float mant = __uint_as_float((bits & 0x007FFFFFu) | 0x3F800000u);
  const float t = __fadd_rn(mant, -1.0f);
  float a = kP6;
  a = __fmaf_rn(a, t, kP5);
  a = __fmaf_rn(a, t, kP4);
  a = __fmaf_rn(a, t, kP3);
  a = __fmaf_rn(a, t, kP2);
  a = __fmaf_rn(a, t, kP1);
  return __fmul_rn(a, t);
}

// 2^e for e <= 0 by nearest-integer range reduction; returns p * 2^i.
__device__ __forceinline__ float ex2_poly(float e) {
  const float ti = __fadd_rn(e, kMagic);          // low mantissa bits = round-half-even(e)
  const float fi = __fadd_rn(ti, -kMagic);
  const float f = __fadd_rn(e, -fi);
  float a = kE4;
  a = __fmaf_rn(a, f, kE3);
  a = __fmaf_rn(a, f, kE2);
  a = __fmaf_rn(a, f, kE1);
  a = __fmaf_rn(a, f, kE0);
  const float p = __fmaf_rn(a, f, 1.0f);
  return __uint_as_float(__float_as_uint(p) + (__float_as_uint(ti) << 23));
}

__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- per-width constants (warp-uniform, set up once per tile) ---------------------------------
struct LinW {
  float invq;    // fl(1/qmax)
  float qmaxf;
  float halff;   // 2^(b-1), the code offset
};
struct LogW {
  float a;       // K/R codes per octave (exact)
  float c;       // fl(R/K) octaves per code
  float negR;    // -R: lowest log-distance that still has a code
  int K;
};
__device__ __forceinline__ LinW lin_width(int b) {
  LinW w;
  const int half = 1 << ((b > 16 ? 16 : b) - 1);
  w.qmaxf = (float)(half - 1);
  w.invq = __fdiv_rn(1.0f, w.qmaxf);
  w.halff = (float)half;
  return w;
}
__device__ __forceinline__ LogW log_width(int b) {
  LogW w;
  const int K = (1 << (b > 16 ? 16 : b)) - 1;
  const int R = K < 30 ? K : 30;
  w.K = K;
  w.a = __fdiv_rn((float)K, (float)R);
  w.c = __fdiv_rn((float)R, (float)K);
  w.negR = -(float)R;
  return w;
}

// ---- raw code words of one lane for one row ---------------------------------------------------
template <bool WIDE>
struct Raw {
  uint32_t w[WIDE ? 4 : 2];
};

// Loads the lane's share of a row's codes.  row_e0 is a multiple of 128; `limit` is the padded
// byte size of the code buffer, so tail rows never read past it.
template <bool WIDE>
__device__ __forceinline__ void load_codes(const uint8_t* base, unsigned long long row_e0, int b,
                                           int lane, unsigned long long limit, Raw<WIDE>& r) {
  r.w[0] = 0u;
  r.w[1] = 0u;
  const unsigned long long rb = (row_e0 >> 3) * (unsigned)b;
  switch (b) {
    case 2: {
      const unsigned long long off = rb + lane;
      if (off < limit) r.w[0] = *(base + off);
    } break;
    case 3: {
      const unsigned long long off = rb + 4 * lane;
      if (lane < 12 && off < limit) r.w[0] = *reinterpret_cast<const uint32_t*>(base + off);
    } break;
    case 4: {
      const unsigned long long off = rb + 2 * lane;
      if (off < limit) r.w[0] = *reinterpret_cast<const uint16_t*>(base + off);
    } break;
    case 8: {
      const unsigned long long off = rb + 4 * lane;
      if (off < limit) r.w[0] = *reinterpret_cast<const uint32_t*>(base + off);
    } break;
    case 16: {
      const unsigned long long off = rb + 8 * lane;
      if (off < limit) {
        const uint2 v = *reinterpret_cast<const uint2*>(base + off);
        r.w[0] = v.x;
        r.w[1] = v.y;
      }
    } break;
    default:
      if constexpr (WIDE) {
        r.w[2] = 0u;
        r.w[3] = 0u;
        const unsigned long long off = rb + 16 * lane;   // b == 32: rb = row_e0 * 4
        if (off < limit) {
          const uint4 v = *reinterpret_cast<const uint4*>(base + off);
          r.w[0] = v.x; r.w[1] = v.y; r.w[2] = v.z; r.w[3] = v.w;
        }
      }
      break;
  }
}

// Splits the lane's raw words into its four codes.  Must be called by the whole warp (the 3-bit
// case exchanges words between lanes).
template <bool WIDE>
__device__ __forceinline__ void split_codes(const Raw<WIDE>& r, int b, int lane, uint32_t (&c)[4]) {
  switch (b) {
    case 2:
#pragma unroll
      for (int k = 0; k < 4; ++k) c[k] = (r.w[0] >> (2 * k)) & 3u;
      break;
    case 3: {
      const int bit = 12 * lane;
      const uint32_t lo = __shfl_sync(kFull, r.w[0], bit >> 5);
      const uint32_t hi = __shfl_sync(kFull, r.w[0], (bit >> 5) + 1);
      const uint32_t f = __funnelshift_r(lo, hi, bit & 31);
#pragma unroll
      for (int k = 0; k < 4; ++k) c[k] = (f >> (3 * k)) & 7u;
    } break;
    case 4:
#pragma unroll
      for (int k = 0; k < 4; ++k) c[k] = (r.w[0] >> (4 * k)) & 15u;
      break;
    case 8:
#pragma unroll
      for (int k = 0; k < 4; ++k) c[k] = (r.w[0] >> (8 * k)) & 255u;
      break;
    case 16:
      c[0] = r.w[0] & 0xFFFFu; c[1] = r.w[0] >> 16;
      c[2] = r.w[1] & 0xFFFFu; c[3] = r.w[1] >> 16;
      break;
    default:
#pragma unroll
      for (int k = 0; k < 4; ++k) c[k] = 0u;
      break;
  }
}

// Packs four values x_k = base + u_k (u_k < 2^b) into the lane's field and stores the row.
// `keep` masks the bits of elements beyond the tensor's end (padding stays zero).
__device__ __forceinline__ void store_codes(uint8_t* base, unsigned long long row_e0, int b, int lane,
                                            unsigned long long limit, const uint32_t (&x)[4],
                                            uint32_t sub, int nvl) {
  const unsigned long long rb = (row_e0 >> 3) * (unsigned)b;
  switch (b) {
    case 2: {
      uint32_t w = x[0] + (x[1] << 2) + (x[2] << 4) + (x[3] << 6) - sub * 85u;
      w &= (1u << (2 * nvl)) - 1u;
      const unsigned long long off = rb + lane;
      if (off < limit) *(base + off) = (uint8_t)w;
    } break;
    case 3: {
      uint32_t p = x[0] + (x[1] << 3) + (x[2] << 6) + (x[3] << 9) - sub * 585u;
      p &= (1u << (3 * nvl)) - 1u;
      // word j of the 48-byte row collects the 12-bit fields that overlap bits [32j, 32j+32)
      const int j = lane;
      const int first = (8 * j) / 3;
      uint32_t w = 0u;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int src = first + i;
        uint32_t v = __shfl_sync(kFull, p, src & 31);
        const int sh = 12 * src - 32 * j;
        if (sh >= 32) v = 0u;
        else if (sh >= 0) v <<= sh;
        else v >>= -sh;
        w |= v;
      }
      const unsigned long long off = rb + 4 * lane;
      if (lane < 12 && off < limit) *reinterpret_cast<uint32_t*>(base + off) = w;
    } break;
    case 4: {
      uint32_t w = x[0] + (x[1] << 4) + (x[2] << 8) + (x[3] << 12) - sub * 4369u;
      w &= (1u << (4 * nvl)) - 1u;
      const unsigned long long off = rb + 2 * lane;
      if (off < limit) *reinterpret_cast<uint16_t*>(base + off) = (uint16_t)w;
    } break;
    case 8: {
      uint32_t w = x[0] + (x[1] << 8) + (x[2] << 16) + (x[3] << 24) - sub * 0x01010101u;
      w &= nvl >= 4 ? 0xFFFFFFFFu : (1u << (8 * nvl)) - 1u;
      const unsigned long long off = rb + 4 * lane;
      if (off < limit) *reinterpret_cast<uint32_t*>(base + off) = w;
    } break;
    case 16: {
      uint32_t w0 = x[0] + (x[1] << 16) - sub * 0x00010001u;
      uint32_t w1 = x[2] + (x[3] << 16) - sub * 0x00010001u;
      w0 &= nvl >= 2 ? 0xFFFFFFFFu : (nvl == 1 ? 0xFFFFu : 0u);
      w1 &= nvl >= 4 ? 0xFFFFFFFFu : (nvl == 3 ? 0xFFFFu : 0u);
      const unsigned long long off = rb + 8 * lane;
      if (off < limit) *reinterpret_cast<uint2*>(base + off) = make_uint2(w0, w1);
    } break;
    default:
      break;
  }
}

__device__ __forceinline__ void store_raw32(uint8_t* base, unsigned long long row_e0, int lane,
                                            unsigned long long limit, const float (&x)[4]) {
  const unsigned long long off = row_e0 * 4 + 16 * lane;
  if (off < limit) *reinterpret_cast<float4*>(base + off) = make_float4(x[0], x[1], x[2], x[3]);
}

__device__ __forceinline__ unsigned long long padded_code_bytes(unsigned long long numel, int b) {
  const unsigned long long by = (numel * (unsigned)b + 7) >> 3;
  return (by + 15) & ~15ull;
}

// ---- variant "sr": stochastic rounding on a grid with a whole number of levels per octave ------------------
__device__ __forceinline__ uint32_t mix32(uint32_t h) {
  h ^= h >> 16; h *= 0x85EBCA6Bu; h ^= h >> 13; h *= 0xC2B2AE35u; h ^= h >> 16;
  return h;
}
__device__ __forceinline__ int sr_lg_levels(int b) { return b == 8 ? 3 : b == 16 ? 11 : 0; }
constexpr float kOnePlus = 0x1.000008p+0f;     // 1 + 2^-21: lifts the block maximum to or just above 1
// c1 = fl(fl(1/s) * (1 + 2^-21)); word: the element's random word
__device__ __forceinline__ uint32_t sr_steps_below(float x, float c1, int b, int K, uint32_t word) {
  const int g = sr_lg_levels(b);
  const int yb = (int)__float_as_uint(__fmul_rn(x, c1));
  int n = 0x3F800000 - yb;
  n = max(n, 0);
  n = min(n, K << (23 - g));
  const unsigned long long j = (((unsigned long long)(uint32_t)n << (9 + g)) + word) >> 32;
  return min((uint32_t)j, (uint32_t)K);
}
__device__ __forceinline__ float sr_level(uint32_t j, int b) {
  return __uint_as_float(0x3F800000u - (j << (23 - sr_lg_levels(b))));
}

// ---- variant "ts": two scales per block --------------------------------------------------------------------
struct TsConst {
  float hi, lo, W, Phi;
  int Ehi;
};
__device__ __forceinline__ float ts_dist(const TsConst& t, uint32_t xb) {
  const float de = (float)((int)(xb >> 23) - t.Ehi);
  const float dp = __fadd_rn(lg_poly(xb), -t.Phi);
  return __fadd_rn(de, dp);
}
__device__ __forceinline__ TsConst ts_consts(float hi, float lo) {
  TsConst t;
  t.hi = hi; t.lo = lo;
  t.Ehi = (int)(__float_as_uint(hi) >> 23);
  t.Phi = lg_poly(__float_as_uint(hi));
  float W = -ts_dist(t, __float_as_uint(lo));
  W = W > 30.0f ? 30.0f : W;
  t.W = W > 0.0f ? W : 0.0f;
  return t;
}
__device__ __forceinline__ float decode_ts(uint32_t c, const TsConst& t, int K) {
  if (t.hi == 0.0f) return 0.0f;
  if (c == 0u) return t.lo;
  const float step = __fdiv_rn(t.W, (float)K);
  const float e = __fmul_rn((float)((int)c - K), step);
  return __fmul_rn(t.hi, ex2_poly(e));
}

// ---- decode ------------------------------------------------------------------------------------
__device__ __forceinline__ float decode_lin(uint32_t c, float s, const LinW& w) {
  const float q = __fadd_rn(__uint_as_float(kTwo23Bits | c), -(kTwo23 + w.halff));
  return __fmul_rn(s, __fmul_rn(q, w.invq));
}
// Variant with the piecewise-linear logarithm (widths 8, 16), in integers: code steps below the
// maximum -> distance in units of the bit pattern, n' = floor(j*B/2^S + 1/2).
__device__ __forceinline__ uint32_t pl_step(int b) { return b == 8 ? 4042322161u : 4026593281u; }   // round(30*2^23*2^S/K)
__device__ __forceinline__ int pl_shift(int b) { return b == 8 ? 12 : 20; }
__device__ __forceinline__ float decode_pl(uint32_t j, uint32_t s_bits, int b) {
  const int S = pl_shift(b);
  const unsigned long long below = ((unsigned long long)j * pl_step(b) + (1ull << (S - 1))) >> S;
  const int xb = (int)s_bits - (int)(uint32_t)below;
  return __uint_as_float((uint32_t)max(xb, 0));
}

// vmode: 0 polynomial logarithm, 1 piecewise-linear (8 and 16 bits), 2 stochastic rounding, 3 two scales (ts)
__device__ __forceinline__ float decode_log(uint32_t c, float s, int b, const LogW& w, unsigned vmode, const TsConst& ts) {
  if (vmode == 2u) return __fmul_rn(s, sr_level((uint32_t)w.K - c, b));
  if (vmode == 3u) return decode_ts(c, ts, w.K);
  if (b <= 4) {   // one octave per code: 2^(c-K)
    return __fmul_rn(s, __uint_as_float((c + (uint32_t)(127 - w.K)) << 23));
  }
  if (vmode == 1u) return decode_pl((uint32_t)w.K - c, __float_as_uint(s), b);
  const float rf = __fadd_rn(__uint_as_float(kTwo23Bits | c), -(kTwo23 + (float)w.K));
  return __fmul_rn(s, ex2_poly(__fmul_rn(rf, w.c)));
}

template <int GDT>
struct GradRow;
template <>
struct GradRow<0> { float4 v; };
template <>
struct GradRow<1> { uint2 v; };
template <>
struct GradRow<2> { uint2 v; };

template <int GDT>
__device__ __forceinline__ void load_grad(const void* grad, unsigned long long e, int nvl, GradRow<GDT>& g) {
  if constexpr (GDT == 0) {
    const float* p = reinterpret_cast<const float*>(grad) + e;
    if (nvl == 4) {
      g.v = __ldg(reinterpret_cast<const float4*>(p));
    } else {
      g.v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (nvl > 0) g.v.x = __ldg(p);
      if (nvl > 1) g.v.y = __ldg(p + 1);
      if (nvl > 2) g.v.z = __ldg(p + 2);
    }
  } else {
    const uint16_t* p = reinterpret_cast<const uint16_t*>(grad) + e;
    if (nvl == 4) {
      g.v = __ldg(reinterpret_cast<const uint2*>(p));
    } else {
      uint32_t a = 0, b = 0, c = 0;
      if (nvl > 0) a = __ldg(p);
      if (nvl > 1) b = __ldg(p + 1);
      if (nvl > 2) c = __ldg(p + 2);
      g.v = make_uint2(a | (b << 16), c);
    }
  }
}
template <int GDT>
__device__ __forceinline__ void widen_grad(const GradRow<GDT>& g, float (&o)[4]) {
  if constexpr (GDT == 0) {
    o[0] = g.v.x; o[1] = g.v.y; o[2] = g.v.z; o[3] = g.v.w;
  } else if constexpr (GDT == 1) {
    o[0] = __uint_as_float(g.v.x << 16);
    o[1] = __uint_as_float(g.v.x & 0xFFFF0000u);
    o[2] = __uint_as_float(g.v.y << 16);
    o[3] = __uint_as_float(g.v.y & 0xFFFF0000u);
  } else {
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&g.v.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&g.v.y));
    o[0] = a.x; o[1] = a.y; o[2] = b.x; o[3] = b.y;
  }
}

// The low-precision copy of up to four updated parameters (nearest-even rounding).
__device__ __forceinline__ void store_param_lp(void* lp, unsigned lp_dtype, unsigned long long e, int nvl,
                                               const float (&x)[4]) {
  uint16_t h[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    if (lp_dtype == 1u) {
      const __nv_bfloat16 b = __float2bfloat16_rn(x[k]);
      h[k] = *reinterpret_cast<const uint16_t*>(&b);
    } else {
      const __half b = __float2half_rn(x[k]);
      h[k] = *reinterpret_cast<const uint16_t*>(&b);
    }
  }
  uint16_t* p = reinterpret_cast<uint16_t*>(lp) + e;
  if (nvl == 4) {
    *reinterpret_cast<uint2*>(p) = make_uint2(h[0] | ((uint32_t)h[1] << 16), h[2] | ((uint32_t)h[3] << 16));
  } else {
    if (nvl > 0) p[0] = h[0];
    if (nvl > 1) p[1] = h[1];
    if (nvl > 2) p[2] = h[2];
  }
}

__device__ __forceinline__ float4 load_param(const float* p, int nvl) {
  if (nvl == 4) return *reinterpret_cast<const float4*>(p);
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (nvl > 0) v.x = p[0];
  if (nvl > 1) v.y = p[1];
  if (nvl > 2) v.z = p[2];
  return v;
}
__device__ __forceinline__ void store_param(float* p, int nvl, const float (&x)[4]) {
  if (nvl == 4) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  } else {
    if (nvl > 0) p[0] = x[0];
    if (nvl > 1) p[1] = x[1];
    if (nvl > 2) p[2] = x[2];
  }
}

// ---- the tile kernel ---------------------------------------------------------------------------
// VAR: the table holds tensors whose second moment uses one of the codes that only this kernel serves
// (stochastic rounding, two scales); compiled apart so that the common launches carry none of it.
template <int MODE, int GDT, bool STATS, bool WIDE, bool VAR>
__global__ void __launch_bounds__(kThreads, 2)
stq_tile_kernel(const TensorDesc* __restrict__ table, const uint32_t* __restrict__ tile_map,
                uint32_t tile_begin, uint32_t tile_end, const StepConsts sc_in, double* __restrict__ partials) {
  StepConsts sc = sc_in;
  if constexpr (MODE == kStep) {
    if (sc_in.dev_scalars != nullptr) {     // step count / learning rate live on the device
      sc.step_size = __ldg(sc_in.dev_scalars + 0);
      sc.rsqrt_bc2 = __ldg(sc_in.dev_scalars + 1);
      sc.lr = (double)__ldg(sc_in.dev_scalars + 2);
    }
  }
  constexpr int R = kRowsPerWarp;
  constexpr bool kHasGrad = (MODE == kStep || MODE == kStatsOnly);
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  float grad_mul = 1.0f;
  if constexpr (MODE == kStep) {
    // a non-finite gradient somewhere in the model: the whole step is skipped
    if (sc.found_inf != nullptr && __ldg(sc.found_inf) != 0.0f) return;
    if (sc.inv_scale != nullptr) grad_mul = __ldg(sc.inv_scale);
  }

  // blocks of 1024 elements: maxima of neighbouring warps meet here (two buffers, used alternately: a warp
  // that runs ahead is held by the next tile's barrier before it can overwrite what a slower one still reads)
  __shared__ uint32_t xchg[2][3 * (kThreads / 32)];      // {max |m|, max v, min v} per warp
  int xchg_parity = 0;

  for (uint32_t tile = tile_begin + blockIdx.x; tile < tile_end; tile += gridDim.x) {
    const TensorDesc* __restrict__ T = table + __ldg(tile_map + tile);
    const unsigned long long numel = T->numel;
    const unsigned long long e_warp =
        (unsigned long long)(T->nfast + (tile - T->tile0s)) * kTile + (unsigned)warp * (R * kRowElems);
    float st_g = 0.f, st_a = 0.f, st_q = 0.f;
    const bool wide_block = MODE != kStatsOnly && T->block == 1024u;

    if (e_warp >= numel && wide_block) {     // nothing to do here, but the neighbour may wait for this warp
      if (lane == 0) {
        xchg[xchg_parity][3 * warp] = 0u; xchg[xchg_parity][3 * warp + 1] = 0u; xchg[xchg_parity][3 * warp + 2] = 0x7F800000u;
      }
      asm volatile("bar.sync 1, %0;" ::"r"(kThreads) : "memory");
    }
    if (e_warp < numel) {
      const uint32_t B = T->block;              // a power of two, 32 .. 1024
      const int lgB = 31 - __clz((int)B);
      const int bm_in = T->bm_in, bv_in = T->bv_in, bm_out = T->bm_out, bv_out = T->bv_out;
      const unsigned vmode = VAR ? T->v_mode : (T->v_mode & 1u);
      const bool pl = vmode == 1u;

      int nvl[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const long long rem = (long long)numel - (long long)(e_warp + r * kRowElems) - 4 * lane;
        nvl[r] = rem >= 4 ? 4 : (rem > 0 ? (int)rem : 0);
      }

      // ---- issue every load of the four rows before anything is consumed -------------------------
      float4 th4[R];
      GradRow<GDT> graw[R];
      Raw<WIDE> rawm[R], rawv[R];
      float s_m_in[R], s_v_in[R];
      [[maybe_unused]] float s_v2_in[R];      // two-scale code: the block minimum
      if constexpr (MODE == kStep) {
        float* param = T->param;
#pragma unroll
        for (int r = 0; r < R; ++r) th4[r] = load_param(param + e_warp + r * kRowElems + 4 * lane, nvl[r]);
      }
      if constexpr (kHasGrad) {
        const void* grad = T->grad;
#pragma unroll
        for (int r = 0; r < R; ++r) load_grad<GDT>(grad, e_warp + r * kRowElems + 4 * lane, nvl[r], graw[r]);
      }
      if constexpr (MODE == kStep || MODE == kRepack) {
        const uint8_t* mc = T->mc_in;
        const uint8_t* vc = T->vc_in;
        const unsigned long long lim_m = padded_code_bytes(numel, bm_in);
        const unsigned long long lim_v = padded_code_bytes(numel, bv_in);
#pragma unroll
        for (int r = 0; r < R; ++r) {
          load_codes<WIDE>(mc, e_warp + r * kRowElems, bm_in, lane, lim_m, rawm[r]);
          load_codes<WIDE>(vc, e_warp + r * kRowElems, bv_in, lane, lim_v, rawv[r]);
        }
        const float* ms = T->ms_in;
        const float* vs = T->vs_in;
#pragma unroll
        for (int r = 0; r < R; ++r) {
          // (blocks of 32 or 64 elements: a row holds several, each lane reads the scale of its own)
          const unsigned long long e_lane = e_warp + r * kRowElems + 4 * lane;
          const bool live = e_lane < numel;
          s_m_in[r] = (live && bm_in != 32) ? ms[e_lane >> lgB] : 0.f;
          if (vmode == 3u) {                  // {hi, lo} per block
            s_v_in[r] = (live && bv_in != 32) ? vs[2 * (e_lane >> lgB)] : 0.f;
            s_v2_in[r] = (live && bv_in != 32) ? vs[2 * (e_lane >> lgB) + 1] : 0.f;
          } else {
            s_v_in[r] = (live && bv_in != 32) ? vs[e_lane >> lgB] : 0.f;
            s_v2_in[r] = 0.f;
          }
        }
      }

      if constexpr (MODE == kStatsOnly) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
          float g[4];
          widen_grad<GDT>(graw[r], g);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            st_g += g[k];
            st_a += fabsf(g[k]);
            st_q = __fmaf_rn(g[k], g[k], st_q);
          }
        }
      } else {
        // ---- decode stored states, form the new moments -----------------------------------------
        float mt[R][4], vt[R][4], th[R][4];
        if constexpr (MODE == kInit) {
#pragma unroll
          for (int r = 0; r < R; ++r)
#pragma unroll
            for (int k = 0; k < 4; ++k) { mt[r][k] = 0.f; vt[r][k] = 0.f; }
        } else {
          const LinW lw_in = lin_width(bm_in);
          const LogW gw_in = log_width(bv_in);
          const float wd = T->wd;
#pragma unroll
          for (int r = 0; r < R; ++r) {
            float mh[4], vh[4];
            if (WIDE && bm_in == 32) {
              if constexpr (WIDE) {
#pragma unroll
                for (int k = 0; k < 4; ++k) mh[k] = __uint_as_float(rawm[r].w[k]);
              }
            } else {
              uint32_t c[4];
              split_codes<WIDE>(rawm[r], bm_in, lane, c);
#pragma unroll
              for (int k = 0; k < 4; ++k) mh[k] = decode_lin(c[k], s_m_in[r], lw_in);
            }
            if (WIDE && bv_in == 32) {
              if constexpr (WIDE) {
#pragma unroll
                for (int k = 0; k < 4; ++k) vh[k] = __uint_as_float(rawv[r].w[k]);
              }
            } else {
              uint32_t c[4];
              split_codes<WIDE>(rawv[r], bv_in, lane, c);
              TsConst ts_in;
              if (vmode == 3u) ts_in = ts_consts(s_v_in[r], s_v2_in[r]);
#pragma unroll
              for (int k = 0; k < 4; ++k) vh[k] = decode_log(c[k], s_v_in[r], bv_in, gw_in, vmode, ts_in);
            }
            if constexpr (MODE == kStep) {
              th[r][0] = th4[r].x; th[r][1] = th4[r].y; th[r][2] = th4[r].z; th[r][3] = th4[r].w;
              float g[4];
              widen_grad<GDT>(graw[r], g);
              if (sc.inv_scale != nullptr) {
#pragma unroll
                for (int k = 0; k < 4; ++k) g[k] = __fmul_rn(g[k], grad_mul);
              }
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                if constexpr (STATS) {
                  st_g += g[k];
                  st_a += fabsf(g[k]);
                  st_q = __fmaf_rn(g[k], g[k], st_q);
                }
                float gk = g[k];
                if (sc.l2_mode) gk = __fadd_rn(gk, __fmul_rn(wd, th[r][k]));
                const float m = __fmaf_rn(sc.b1, mh[k], __fmul_rn(sc.c1, gk));
                const float v = __fmaf_rn(sc.b2, vh[k], __fmul_rn(__fmul_rn(sc.c2, gk), gk));
                // elements past the end of the tensor stay out of the block maximum
                mt[r][k] = k < nvl[r] ? m : 0.f;
                vt[r][k] = k < nvl[r] ? v : 0.f;
              }
            } else {   // kRepack: the stored values themselves are re-quantized
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                mt[r][k] = k < nvl[r] ? mh[k] : 0.f;
                vt[r][k] = k < nvl[r] ? vh[k] : 0.f;
              }
            }
          }
        }

        // ---- block maxima: lane max of 4, warp REDUX on the bit patterns, rows merged per block ----
        uint32_t mxm[R], mxv[R];
        [[maybe_unused]] uint32_t mnv[R];     // two-scale code: block minimum of v (elements past the end stay out)
        // lanes that share a block with this one: the whole warp, or 8 / 16 neighbours for blocks of 32 / 64
        const unsigned seg_lanes = B >= 128 ? 32u : B / 4;
        const unsigned seg_mask = B >= 128 ? kFull : ((1u << seg_lanes) - 1u) << (lane & ~(seg_lanes - 1u));
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const float am = fmaxf(fmaxf(fabsf(mt[r][0]), fabsf(mt[r][1])), fmaxf(fabsf(mt[r][2]), fabsf(mt[r][3])));
          const float av = fmaxf(fmaxf(vt[r][0], vt[r][1]), fmaxf(vt[r][2], vt[r][3]));
          mxm[r] = __reduce_max_sync(seg_mask, __float_as_uint(am));
          mxv[r] = __reduce_max_sync(seg_mask, __float_as_uint(av));
          mnv[r] = 0x7F800000u;
          if (vmode == 3u) {
            uint32_t lm = 0x7F800000u;
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (k < nvl[r]) lm = min(lm, __float_as_uint(vt[r][k]));
            mnv[r] = __reduce_min_sync(seg_mask, lm);
          }
        }
        if (B >= 256) {
#pragma unroll
          for (int r = 0; r < R; r += 2) {
            mxm[r] = mxm[r + 1] = max(mxm[r], mxm[r + 1]);
            mxv[r] = mxv[r + 1] = max(mxv[r], mxv[r + 1]);
            mnv[r] = mnv[r + 1] = min(mnv[r], mnv[r + 1]);
          }
        }
        if (R >= 4 && B >= 512) {
          const uint32_t a = max(mxm[0], mxm[R - 2]), b = max(mxv[0], mxv[R - 2]), c = min(mnv[0], mnv[R - 2]);
#pragma unroll
          for (int r = 0; r < R; ++r) { mxm[r] = a; mxv[r] = b; mnv[r] = c; }
        }
        if (B == 1024) {
          // a block of 1024 spans this warp and its neighbour: the two exchange their maxima through shared
          // memory.  Every warp of the CTA takes part in the barrier (the ones past the end of the tensor from
          // the branch below), which the whole CTA reaches because the block size is a property of the tile.
          uint32_t* slot = xchg[xchg_parity];
          if (lane == 0) { slot[3 * warp] = mxm[0]; slot[3 * warp + 1] = mxv[0]; slot[3 * warp + 2] = mnv[0]; }
          asm volatile("bar.sync 1, %0;" ::"r"(kThreads) : "memory");
          const uint32_t pm = slot[3 * (warp ^ 1)], pv = slot[3 * (warp ^ 1) + 1], pn = slot[3 * (warp ^ 1) + 2];
#pragma unroll
          for (int r = 0; r < R; ++r) { mxm[r] = max(mxm[r], pm); mxv[r] = max(mxv[r], pv); mnv[r] = min(mnv[r], pn); }
        }

        // ---- quantize, pack, store; decode the new codes; update the parameters -------------------
        const LinW lw = lin_width(bm_out);
        const LogW gw = log_width(bv_out);
        const unsigned long long lim_mo = padded_code_bytes(numel, bm_out);
        const unsigned long long lim_vo = padded_code_bytes(numel, bv_out);
        uint8_t* mco = T->mc_out;
        uint8_t* vco = T->vc_out;
        float* mso = T->ms_out;
        float* vso = T->vs_out;
        float* param = T->param;
        // decoupled decay as theta - (theta*lr*wd + update): the small term keeps its own precision
        // (a factor 1 - lr*wd rounded to fp32 is off by ~1e-3 of the decay it applies)
        const float lrwd = sc.l2_mode ? 0.0f : (float)(sc.lr * (double)T->wd);
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const unsigned long long e_row = e_warp + r * kRowElems;
          if (e_row >= numel) break;
          float mq[4], vq[4];

          // first moment, linear symmetric
          if (WIDE && bm_out == 32) {
            if constexpr (WIDE) {
              store_raw32(mco, e_row, lane, lim_mo, mt[r]);
#pragma unroll
              for (int k = 0; k < 4; ++k) mq[k] = mt[r][k];
            }
          } else {
            const float s_raw = __uint_as_float(mxm[r]);
            const bool zero = s_raw < kTiny;
            const float s = zero ? 0.f : s_raw;
            const float inv = zero ? 0.f : __fmul_rn(lw.qmaxf, __frcp_rn(s_raw));
            const float mg = kMagic + lw.halff;
            uint32_t x[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float t = __fmaf_rn(mt[r][k], inv, mg);    // low bits: q + 2^(b-1)
              x[k] = __float_as_uint(t);
              mq[k] = __fmul_rn(s, __fmul_rn(__fadd_rn(t, -mg), lw.invq));
            }
            store_codes(mco, e_row, bm_out, lane, lim_mo, x, kMagicBits, nvl[r]);
            if (((e_row + 4 * lane) & (B - 1)) == 0 && e_row + 4 * lane < numel) mso[(e_row + 4 * lane) >> lgB] = s;
          }

          // second moment, logarithmic
          if (WIDE && bv_out == 32) {
            if constexpr (WIDE) {
              store_raw32(vco, e_row, lane, lim_vo, vt[r]);
#pragma unroll
              for (int k = 0; k < 4; ++k) vq[k] = vt[r][k];
            }
          } else {
            const float s_raw = __uint_as_float(mxv[r]);
            const bool zero = s_raw < kTiny;
            const float s = zero ? 0.f : s_raw;
            uint32_t x[4];
            uint32_t sub;
            if (vmode == 2u) {
              // stochastic rounding: j = floor(n * L / 2^23 + U / 2^32) level steps below the maximum, U the
              // element's random word (a re-pack has no step to draw from and rounds to nearest)
              const float c1 = zero ? 0.f : __fmul_rn(__frcp_rn(s_raw), kOnePlus);
              uint32_t key_e = 0u;
              if constexpr (MODE == kStep) key_e = mix32(mix32(T->sr_id ^ sc.sr_h) + (uint32_t)(e_row >> 32));
              sub = 0u;
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                uint32_t word = 0x80000000u;
                if constexpr (MODE == kStep) word = mix32(((uint32_t)e_row + 4u * lane + k) ^ key_e);
                const uint32_t j = zero ? (uint32_t)gw.K : sr_steps_below(vt[r][k], c1, bv_out, gw.K, word);
                x[k] = (uint32_t)gw.K - j;
                if constexpr (MODE == kStep) vq[k] = __fmul_rn(s, sr_level(j, bv_out));
              }
            } else if (vmode == 3u) {
              // two scales: codes spread evenly in log2 between the block minimum (raised to hi * 2^-30) and maximum
              const float lo = zero ? 0.f : fmaxf(__uint_as_float(mnv[r]), __fmul_rn(s_raw, 0x1p-30f));
              const TsConst ts = ts_consts(zero ? 1.0f : s_raw, zero ? 1.0f : lo);
              const float inv = ts.W > 0.0f ? __fdiv_rn((float)gw.K, ts.W) : 0.0f;
              sub = kMagicBits - (uint32_t)gw.K;
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const float d = fminf(fmaxf(ts_dist(ts, __float_as_uint(vt[r][k])), -ts.W), 0.0f);
                const float t = __fmaf_rn(d, inv, kMagic);        // low bits: code - K, in [-K, 0]
                x[k] = zero ? sub : __float_as_uint(t);
                if constexpr (MODE == kStep) {
                  TsConst td = ts;
                  td.hi = s;          // (a zero block decodes to zero)
                  vq[k] = decode_ts(x[k] - sub, td, gw.K);
                }
              }
              if (((e_row + 4 * lane) & (B - 1)) == 0 && e_row + 4 * lane < numel) vso[2 * ((e_row + 4 * lane) >> lgB) + 1] = lo;
            } else if (bv_out <= 4) {
              // one octave per code: the code is the exponent of x*sqrt2/s, floored at -K
              const float c = zero ? 0.f : __fmul_rn(__frcp_rn(s_raw), kSqrt2);
              const float ymin = __uint_as_float((uint32_t)(127 - gw.K) << 23);
              sub = (uint32_t)(127 - gw.K);
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const uint32_t yb = __float_as_uint(fmaxf(__fmul_rn(vt[r][k], c), ymin));
                x[k] = yb >> 23;
                if constexpr (MODE == kStep) vq[k] = __fmul_rn(s, __uint_as_float(yb & 0x7F800000u));
              }
            } else if (pl) {
              // distance below the block maximum in units of the bit pattern, at most 30 octaves;
              // j = floor(n*K/D + 1/2) = (n * (512*K/30) + 2^31) >> 32, the factor being a whole number
              const uint32_t s_enc = zero ? 0x7F800000u : mxv[r];     // zero block: every code is the floor
              const uint32_t s_dec = zero ? 0u : mxv[r];
              const uint32_t A = bv_out == 8 ? 4352u : 1118464u;
              sub = 0u;
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const uint32_t n = min(s_enc - __float_as_uint(vt[r][k]), 30u << 23);
                const uint32_t j = (uint32_t)(((unsigned long long)n * A + (1ull << 31)) >> 32);
                x[k] = (uint32_t)gw.K - j;
                if constexpr (MODE == kStep) vq[k] = decode_pl(j, s_dec, bv_out);
              }
            } else {
              const int Es = zero ? kZeroBlockExp : (int)(mxv[r] >> 23);
              const float Ps = lg_poly(mxv[r]);
              const uint32_t ebase = kMagicBits - (uint32_t)Es;
              sub = kMagicBits - (uint32_t)gw.K;
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const uint32_t xb = __float_as_uint(vt[r][k]);
                const float de = __fadd_rn(__uint_as_float(ebase + (xb >> 23)), -kMagic);   // float(E_x - E_s)
                const float dp = __fadd_rn(lg_poly(xb), -Ps);
                const float d = fmaxf(__fadd_rn(de, dp), gw.negR);
                const float t = __fmaf_rn(d, gw.a, kMagic);       // low bits: code - K, in [-K, 0]
                x[k] = __float_as_uint(t);
                if constexpr (MODE == kStep)
                  vq[k] = __fmul_rn(s, ex2_poly(__fmul_rn(__fadd_rn(t, -kMagic), gw.c)));
              }
            }
            store_codes(vco, e_row, bv_out, lane, lim_vo, x, sub, nvl[r]);
            if (((e_row + 4 * lane) & (B - 1)) == 0 && e_row + 4 * lane < numel)
              vso[vmode == 3u ? 2 * ((e_row + 4 * lane) >> lgB) : (e_row + 4 * lane) >> lgB] = s;
          }

          if constexpr (MODE == kStep) {
            float out[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float den = __fmaf_rn(sqrt_approx(vq[k]), sc.rsqrt_bc2, sc.eps);
              const float upd = __fdividef(__fmul_rn(mq[k], sc.step_size), den);
              out[k] = __fadd_rn(th[r][k], -__fmaf_rn(th[r][k], lrwd, upd));
            }
            store_param(param + e_row + 4 * lane, nvl[r], out);
            if (T->param_lp != nullptr) store_param_lp(T->param_lp, T->lp_dtype, e_row + 4 * lane, nvl[r], out);
          }
        }
      }
    }

    if (wide_block) xchg_parity ^= 1;
    if constexpr (STATS || MODE == kStatsOnly) {
      // one partial per warp and tile; the finishing kernel adds them in a fixed order
      double dg = (double)st_g, da = (double)st_a, dq = (double)st_q;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        dg += __shfl_down_sync(kFull, dg, o);
        da += __shfl_down_sync(kFull, da, o);
        dq += __shfl_down_sync(kFull, dq, o);
      }
      if (lane == 0) {
        double* p = partials + ((size_t)tile * (kThreads / 32) + warp) * 3;
        p[0] = dg; p[1] = da; p[2] = dq;
      }
    }
  }
}

// Statistics alone (Algorithm 1 takes them before the update): a streaming reduction over the
// gradients.  Same tile order and the same slots of partial sums as the fused path (eight per tile, one per
// warp there), so the second stage is shared; here ONE warp takes 8 KB of a tile (all of it with 16-bit
// gradients, half with fp32), fills the first of its slots and zeroes the rest: the work that is not arithmetic
// on the elements (finding the tile, the butterfly, the store) is then paid once per 8 KB and not once per
// 1 KB, which keeps the pass bound by memory and not by instruction issue.  A lane reads 128-bit words at a
// 512-byte warp stride.
constexpr uint32_t kGradStatsTilesPerCta = kThreads / 32;     // shares a CTA takes per turn: one per warp

template <int GDT>
__device__ __forceinline__ void grad_stats_accumulate(const uint4& raw, float2& a0, float& a1x, float& a1y, float2& a2) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
  if constexpr (GDT == 0) {
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const float2 g = make_float2(__uint_as_float(w[2 * k]), __uint_as_float(w[2 * k + 1]));
      a0 = __fadd2_rn(a0, g);
      a1x += fabsf(g.x);
      a1y += fabsf(g.y);
      a2 = __ffma2_rn(g, g, a2);
    }
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float2 g;
      if constexpr (GDT == 1) g = make_float2(__uint_as_float(w[k] << 16), __uint_as_float(w[k] & 0xFFFF0000u));
      else g = __half22float2(*reinterpret_cast<const __half2*>(&w[k]));
      a0 = __fadd2_rn(a0, g);
      a1x += fabsf(g.x);
      a1y += fabsf(g.y);
      a2 = __ffma2_rn(g, g, a2);
    }
  }
}

// warps per tile: a warp's share is 8 KB of gradients whatever their type
__host__ __device__ constexpr uint32_t grad_stats_split(int gdt) { return gdt == 0 ? 2u : 1u; }

template <int GDT>
__global__ void __launch_bounds__(kThreads)
stq_grad_stats_kernel(const TensorDesc* __restrict__ table, const uint32_t* __restrict__ tile_map,
                      uint32_t tile_begin, uint32_t tile_end, double* __restrict__ partials) {
  constexpr int kPerLoad = GDT == 0 ? 4 : 8;                 // elements per 128-bit load
  constexpr uint32_t kSplit = grad_stats_split(GDT);
  constexpr uint32_t kShare = kTile / kSplit;                // elements a warp takes
  constexpr int kLoads = kShare / (32 * kPerLoad);           // loads per lane and share
  constexpr int kBatch = 8;                                  // of which in flight together
  constexpr uint32_t kSlots = (kThreads / 32) * 3;           // doubles per tile in `partials`
  constexpr uint32_t kMine = kSlots / kSplit;                // of which this warp writes
  static_assert(kLoads % kBatch == 0, "whole batches");
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned long long n_shares = (unsigned long long)(tile_end - tile_begin) * kSplit;
  const unsigned long long stride = (unsigned long long)gridDim.x * kGradStatsTilesPerCta;
  for (unsigned long long u = (unsigned long long)blockIdx.x * kGradStatsTilesPerCta + (unsigned)warp; u < n_shares; u += stride) {
    const uint32_t tile = tile_begin + (uint32_t)(u / kSplit), part = (uint32_t)(u % kSplit);
    const TensorDesc* __restrict__ T = table + __ldg(tile_map + tile);
    const unsigned long long numel = T->numel;
    const unsigned long long e0 = (unsigned long long)(T->nfast + (tile - T->tile0s)) * kTile + part * kShare;
    const uint8_t* __restrict__ base = reinterpret_cast<const uint8_t*>(T->grad) + e0 * (GDT == 0 ? 4 : 2);
    float2 a0 = make_float2(0.f, 0.f), a2 = make_float2(0.f, 0.f);
    float a1x = 0.f, a1y = 0.f;
    if (e0 + kShare <= numel) {
      const uint4* __restrict__ src = reinterpret_cast<const uint4*>(base) + lane;
#pragma unroll 1
      for (int b = 0; b < kLoads / kBatch; ++b) {
        uint4 raw[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) raw[j] = __ldg(src + (b * kBatch + j) * 32);
#pragma unroll
        for (int j = 0; j < kBatch; ++j) grad_stats_accumulate<GDT>(raw[j], a0, a1x, a1y, a2);
      }
    } else if (e0 < numel) {   // the ragged end of a tensor: whole words while they last, then element by element
#pragma unroll 1
      for (int j = 0; j < kLoads; ++j) {
        const unsigned long long e = e0 + (unsigned long long)(j * 32 + lane) * kPerLoad;
        uint4 raw = make_uint4(0u, 0u, 0u, 0u);
        if (e + kPerLoad <= numel) {
          raw = __ldg(reinterpret_cast<const uint4*>(base) + j * 32 + lane);
        } else if (e < numel) {
          uint32_t w[4] = {0u, 0u, 0u, 0u};
          for (int k = 0; k < kPerLoad && e + k < numel; ++k) {
            if constexpr (GDT == 0) w[k] = __float_as_uint(__ldg(reinterpret_cast<const float*>(T->grad) + e + k));
            else w[k >> 1] |= (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(T->grad) + e + k) << (16 * (k & 1));
          }
          raw = make_uint4(w[0], w[1], w[2], w[3]);
        }
        grad_stats_accumulate<GDT>(raw, a0, a1x, a1y, a2);
      }
    }
    // pairwise butterfly that spreads the three sums over the lanes on the way down: they end in lanes 0, 8, 16
    const float s0 = a0.x + a0.y, s1 = a1x + a1y, s2 = a2.x + a2.y;
    const bool hi = lane & 16;
    float x = (hi ? s2 : s0) + __shfl_xor_sync(kFull, hi ? s0 : s2, 16);
    float y = (hi ? 0.f : s1) + __shfl_xor_sync(kFull, hi ? s1 : 0.f, 16);
    const bool q = lane & 8;
    float z = (q ? y : x) + __shfl_xor_sync(kFull, q ? x : y, 8);
    z += __shfl_xor_sync(kFull, z, 4);
    z += __shfl_xor_sync(kFull, z, 2);
    z += __shfl_xor_sync(kFull, z, 1);
    const float mine = __shfl_sync(kFull, z, (lane & 3) * 8);
    // this warp's slots of the tile: its three sums, then zeros
    if (lane < (int)kMine) partials[(size_t)tile * kSlots + part * kMine + lane] = lane < 3 ? (double)mine : 0.0;
  }
}

// Statistics, second stage, step 1: one CTA per segment of kStatSegTiles tiles of one tensor.
__global__ void __launch_bounds__(256)
stq_stats_segment_kernel(const TensorDesc* __restrict__ table, const uint32_t* __restrict__ seg_map, uint32_t n_seg,
                         const double* __restrict__ partials, double* __restrict__ seg_sums) {
  constexpr uint32_t W = kThreads / 32;   // partials per tile
  const uint32_t sidx = blockIdx.x;
  if (sidx >= n_seg) return;
  const TensorDesc* T = table + seg_map[sidx];
  const uint32_t j = sidx - T->seg0;                       // segment number inside the tensor
  const uint32_t nt = T->nfast + T->nslow;
  const uint32_t first = j * kStatSegTiles;
  const uint32_t count = min((uint32_t)kStatSegTiles, nt - first) * W;
  double a[3] = {0.0, 0.0, 0.0};
  for (uint32_t i = threadIdx.x; i < count; i += blockDim.x) {
    const uint32_t ti = first + i / W;
    const size_t t = ti < T->nfast ? (size_t)T->tile0 + ti : (size_t)T->tile0s + (ti - T->nfast);
#pragma unroll
    for (int k = 0; k < 3; ++k) a[k] += partials[(t * W + (i % W)) * 3 + k];
  }
  __shared__ double sh[256][3];
#pragma unroll
  for (int k = 0; k < 3; ++k) sh[threadIdx.x][k] = a[k];
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) {
#pragma unroll
      for (int k = 0; k < 3; ++k) sh[threadIdx.x][k] += sh[threadIdx.x + s][k];
    }
    __syncthreads();
  }
  if (threadIdx.x < 3) seg_sums[(size_t)sidx * 3 + threadIdx.x] = sh[0][threadIdx.x];
}

// Step 2: one CTA per tensor adds its segments.
__global__ void __launch_bounds__(256)
stq_stats_finish_kernel(const TensorDesc* __restrict__ table, int L, const double* __restrict__ seg_sums,
                        double* __restrict__ out) {
  const int l = blockIdx.x;
  if (l >= L) return;
  const uint32_t nt = table[l].nfast + table[l].nslow;
  const uint32_t ns = (nt + kStatSegTiles - 1) / kStatSegTiles, s0 = table[l].seg0;
  double a[3] = {0.0, 0.0, 0.0};
  for (uint32_t i = threadIdx.x; i < ns; i += blockDim.x) {
#pragma unroll
    for (int k = 0; k < 3; ++k) a[k] += seg_sums[(size_t)(s0 + i) * 3 + k];
  }
  __shared__ double sh[256][3];
#pragma unroll
  for (int k = 0; k < 3; ++k) sh[threadIdx.x][k] = a[k];
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) {
#pragma unroll
      for (int k = 0; k < 3; ++k) sh[threadIdx.x][k] += sh[threadIdx.x + s][k];
    }
    __syncthreads();
  }
  if (threadIdx.x < 3) out[(size_t)l * 4 + threadIdx.x] = sh[0][threadIdx.x];
  if (threadIdx.x == 3) out[(size_t)l * 4 + 3] = (double)table[l].numel;
}

template <int MODE, int GDT, bool STATS, bool WIDE, bool VAR>
cudaError_t launch_one(const TensorDesc* table, const uint32_t* tile_map, uint32_t tb, uint32_t te,
                       const StepConsts& sc, double* partials, int grid, cudaStream_t stream) {
  const uint32_t n = te - tb;
  const int g = (int)(n < (uint32_t)grid ? n : (uint32_t)grid);
  stq_tile_kernel<MODE, GDT, STATS, WIDE, VAR><<<g, kThreads, 0, stream>>>(table, tile_map, tb, te, sc, partials);
  return cudaGetLastError();
}

template <int MODE, int GDT, bool STATS>
cudaError_t launch_w(bool wide, const TensorDesc* table, const uint32_t* tile_map, uint32_t tb, uint32_t te,
                     const StepConsts& sc, double* partials, int grid, cudaStream_t stream, bool variants) {
  if (variants)
    return wide ? launch_one<MODE, GDT, STATS, true, true>(table, tile_map, tb, te, sc, partials, grid, stream)
                : launch_one<MODE, GDT, STATS, false, true>(table, tile_map, tb, te, sc, partials, grid, stream);
  return wide ? launch_one<MODE, GDT, STATS, true, false>(table, tile_map, tb, te, sc, partials, grid, stream)
              : launch_one<MODE, GDT, STATS, false, false>(table, tile_map, tb, te, sc, partials, grid, stream);
}

}  // namespace

cudaError_t launch_tiles(Mode mode, bool wide, bool variants, int grad_dtype, bool stats, const TensorDesc* table,
                         const uint32_t* tile_map, uint32_t tile_begin, uint32_t tile_end,
                         const StepConsts& sc, double* partials, int grid, cudaStream_t stream) {
  if (tile_end <= tile_begin) return cudaSuccess;
  switch (mode) {
    case kStep:
      if (grad_dtype == 0)
        return stats ? launch_w<kStep, 0, true>(wide, table, tile_map, tile_begin, tile_end, sc, partials, grid, stream, variants)
                     : launch_w<kStep, 0, false>(wide, table, tile_map, tile_begin, tile_end, sc, partials, grid, stream, variants);
      if (grad_dtype == 1)
        return stats ? launch_w<kStep, 1, true>(wide, table, tile_map, tile_begin, tile_end, sc, partials, grid, stream, variants)
                     : launch_w<kStep, 1, false>(wide, table, tile_map, tile_begin, tile_end, sc, partials, grid, stream, variants);
      return stats ? launch_w<kStep, 2, true>(wide, table, tile_map, tile_begin, tile_end, sc, partials, grid, stream, variants)
                   : launch_w<kStep, 2, false>(wide, table, tile_map, tile_begin, tile_end, sc, partials, grid, stream, variants);
    case kRepack:
      return launch_w<kRepack, 0, false>(wide, table, tile_map, tile_begin, tile_end, sc, partials, grid, stream, variants);
    case kInit:
      return launch_w<kInit, 0, false>(wide, table, tile_map, tile_begin, tile_end, sc, partials, grid, stream, variants);
    case kStatsOnly: {
      const uint32_t n = tile_end - tile_begin;
      const uint32_t want = (uint32_t)grid * 4u;   // small CTAs of few registers: many fit per SM
      // a warp takes 8 KB of gradients per turn
      const uint32_t need = (uint32_t)(((unsigned long long)n * grad_stats_split(grad_dtype) + kGradStatsTilesPerCta - 1u) / kGradStatsTilesPerCta);
      // every CTA gets the same number of turns (a short launch of uneven turns would end on a few stragglers)
      const uint32_t turns = (need + want - 1u) / want;
      const int g = (int)((need + turns - 1u) / turns);
      if (grad_dtype == 0)
        stq_grad_stats_kernel<0><<<g, kThreads, 0, stream>>>(table, tile_map, tile_begin, tile_end, partials);
      else if (grad_dtype == 1)
        stq_grad_stats_kernel<1><<<g, kThreads, 0, stream>>>(table, tile_map, tile_begin, tile_end, partials);
      else
        stq_grad_stats_kernel<2><<<g, kThreads, 0, stream>>>(table, tile_map, tile_begin, tile_end, partials);
      return cudaGetLastError();
    }
  }
  return cudaErrorInvalidValue;
}

cudaError_t launch_stats_finish(const TensorDesc* table, int L, const uint32_t* seg_map, uint32_t n_seg,
                                const double* partials, double* seg_sums, double* out, cudaStream_t stream) {
  stq_stats_segment_kernel<<<n_seg, 256, 0, stream>>>(table, seg_map, n_seg, partials, seg_sums);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  stq_stats_finish_kernel<<<L, 256, 0, stream>>>(table, L, seg_sums, out);
  return cudaGetLastError();
}

__global__ void stq_step_scalars_kernel(const long long* __restrict__ step_dev, const float* __restrict__ lr_dev,
                                        double lr_host, double beta1, double beta2, float* __restrict__ out) {
  long long t = *step_dev;
  if (t < 1) t = 1;
  const double lr = lr_dev != nullptr ? (double)*lr_dev : lr_host;
  const double bc1 = 1.0 - pow(beta1, (double)t);
  const double bc2 = 1.0 - pow(beta2, (double)t);
  out[0] = (float)(lr / bc1);
  out[1] = (float)(1.0 / sqrt(bc2));
  out[2] = (float)lr;
}

cudaError_t launch_step_scalars(const long long* step_dev, const float* lr_dev, double lr_host, double beta1,
                                double beta2, float* out, cudaStream_t stream) {
  stq_step_scalars_kernel<<<1, 1, 0, stream>>>(step_dev, lr_dev, lr_host, beta1, beta2, out);
  return cudaGetLastError();
}

__global__ void stq_stats_valid_kernel(const float* __restrict__ found_inf, int* __restrict__ valid) {
  *valid = (found_inf == nullptr || *found_inf == 0.0f) ? 1 : 0;
}

cudaError_t launch_stats_valid(const float* found_inf, int* valid, cudaStream_t stream) {
  stq_stats_valid_kernel<<<1, 1, 0, stream>>>(found_inf, valid);
  return cudaGetLastError();
}

int step_ctas_per_sm() {
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, stq_tile_kernel<kStep, 1, false, false, false>, kThreads, 0) !=
      cudaSuccess)
    return 1;
  return n > 0 ? n : 1;
}

}  // namespace stq

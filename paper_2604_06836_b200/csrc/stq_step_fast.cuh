// The main kernel of the quantized AdamW step: full tiles of tensors with packed states (2..16 bits)
// on both sides of the step.  Tensors that keep their widths run bodies fused and specialised on the
// width pair; tensors that change width inside the step run one runtime-width body in a second launch
// (template flag SPLIT).  Everything else (ragged last tiles, 32-bit states, block 512, init, repack)
// goes through the generic kernel in stq_kernels.cu.
//
// Data movement: a persistent CTA walks its tiles through a shared-memory ring.  A producer warp
// (one elected lane) runs ahead: per tile it writes a small descriptor and issues six bulk
// asynchronous copies (parameters, gradients, m codes, v codes, m scales, v scales: each a contiguous,
// 16-byte aligned range because a tile starts at a multiple of 4096 elements) that complete on the
// stage's "full" mbarrier.  The eight consumer warps never synchronise with each other: each waits
// on "full", pulls its rows into registers with conflict-free 128/64/32-bit shared loads, arrives on
// the stage's "empty" mbarrier (which lets the producer refill it) and computes.  Results go
// straight from registers to global memory with 128-bit (parameters) and 8..64-bit (codes) stores.
// Every wait on a barrier is bounded; on expiry the kernel raises an error flag and returns.
//
// Arithmetic: identical to the generic kernel (same roundings, see there).  The whole tile body is
// specialised on the pair of widths (one dispatch per tile), so shifts and masks are immediates;
// the per-block constants (a reciprocal or a logarithm of the block maximum) are computed by one
// lane per row and broadcast.
// (This header is the kernel itself; it is compiled into several translation units, one per work list, so that the
// instantiations build side by side.  Everything lives in an unnamed namespace: each unit has its own copy.)
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "stq_internal.h"

namespace stq {
namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23
constexpr uint32_t kMagicBits = 0x4B400000u;
constexpr float kTwo23 = 8388608.0f;
constexpr uint32_t kTwo23Bits = 0x4B000000u;
constexpr float kTiny = 0x1p-100f;
constexpr int kZeroBlockExp = 1 << 20;
constexpr float kSqrt2 = 0x1.6a09e6p+0f;

constexpr float kP1 = 0x1.714b30p+0f, kP2 = -0x1.6fc360p-1f, kP3 = 0x1.d54a42p-2f,
                kP4 = -0x1.1e4792p-2f, kP5 = 0x1.f9c008p-4f, kP6 = -0x1.b19412p-6f;
constexpr float kE0 = 0x1.62e42ap-1f, kE1 = 0x1.ebf9bcp-3f, kE2 = 0x1.c6b74cp-5f,
                kE3 = 0x1.3cea84p-7f, kE4 = 0x1.5bbc6ap-10f;

constexpr int R = kRowsPerWarp;
constexpr int kStages = kFastStages;
constexpr int kConsumerWarps = kThreads / 32;
constexpr int kFastThreads = kThreads + 32;      // + the producer warp
constexpr int kOffTheta = 0;
constexpr int kOffGrad = 4 * kTile;
constexpr int kOffMc = 8 * kTile;
constexpr int kOffVc = 10 * kTile;
constexpr int kScaleBytes = (kTile / 128) * 4;   // block scales of one state of the tile, at most
constexpr int kOffMs = 12 * kTile;
constexpr int kOffVs = kOffMs + kScaleBytes;       // (the two-scale code of v keeps two floats per block)
constexpr int kStageBytes = 12 * kTile + 3 * kScaleBytes;
static_assert(kScaleBytes % 16 == 0 && kStageBytes % 128 == 0, "bulk copies need 16-byte aligned destinations");

// What the consumers need to know about a staged tile; written by the producer.
struct __align__(16) TileInfo {
  float* param;        // all pointers are already advanced to the tile's first element / block
  uint8_t* mco;
  uint8_t* vco;
  float* mso;
  float* vso;
  uint16_t* lp;        // low-precision copy of the parameters (2 bytes per element), or nullptr
  uint32_t packed;     // width index of m | of v << 8 (0..4 for 2,3,4,8,16 bits; 5, 6: 8, 16 bits in the
                       // piecewise-linear variant) | log2(block) << 16 | lp dtype << 24
  float wdx;           // fp32(lr*wd) (AdamW) or fp32(wd) (L2 mode)
  uint32_t tile;       // index of the tile in the launch's tile order; 0xFFFFFFFF closes the stream
  uint32_t out;        // width indices to write, m | v << 8 (same coding); equal to the low half of `packed`
                       // unless the step changes the widths of this tensor
  uint32_t sr_key;     // stochastic rounding: mix32(key of the tensor + high word of the element index)
  uint32_t e0;         // low word of the index (inside its tensor) of the tile's first element
  uint32_t pad[2];
};
constexpr int kInfoBytes = 80;
static_assert(sizeof(TileInfo) == kInfoBytes, "TileInfo is read with five 128-bit loads");

constexpr int kOffInfo = kStages * kStageBytes;
constexpr int kOffBars = kOffInfo + kStages * kInfoBytes;        // full[kStages], empty[kStages]
constexpr int kOffLut = kOffBars + 16 * kStages;         // 256 floats: decode table of the 8-bit log code, then
constexpr int kSmemBytes = kOffLut + 2048;               // 256 integers: the same for its piecewise-linear variant
constexpr long long kWaitCycles = 4000000000ll;   // ~2 s: far beyond any copy; then give up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: returns false if the phase did not complete within `limit` cycles.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, long long limit = kWaitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > limit) return false;
  }
  return true;
}
// 1-D bulk copy global -> shared of this CTA, completion counted in bytes on `bar`.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// the mixing function of the stochastic-rounding code (a bijection of the 32-bit words)
__device__ __forceinline__ uint32_t mix32(uint32_t h) {
  h ^= h >> 16; h *= 0x85EBCA6Bu; h ^= h >> 13; h *= 0xC2B2AE35u; h ^= h >> 16;
  return h;
}

__device__ __forceinline__ float sqrt_fast(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_fast(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

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
__device__ __forceinline__ float ex2_poly(float e) {
  const float ti = __fadd_rn(e, kMagic);
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

// ---- per-width constants --------------------------------------------------------------------------
template <int B>
struct Wd {
  static constexpr int half = 1 << (B - 1);
  static constexpr int qmax = half - 1;
  static constexpr int K = (1 << B) - 1;
  static constexpr int Roct = K < 30 ? K : 30;
  static constexpr uint32_t mask = (uint32_t)K;
  static constexpr uint32_t emin = (uint32_t)(127 - K);   // exponent field of the octave floor level
  // sum_k 2^(k*B) over the elements packed into one 32-bit word
  static constexpr uint32_t fieldsum = B == 2 ? 85u : B == 3 ? 585u : B == 4 ? 4369u : B == 8 ? 0x01010101u : 0x00010001u;
};

// The lane's raw code words of one row, read from the staged tile.  row_base: byte address of the
// row's codes in shared memory (row * 16 * B).
template <int B>
__device__ __forceinline__ void lds_codes(const uint8_t* row_base, int lane, uint32_t (&w)[2]) {
  w[1] = 0u;
  if constexpr (B == 2) {
    w[0] = *(row_base + lane);
  } else if constexpr (B == 3) {
    const int bit = 12 * lane;
    const uint32_t* p = reinterpret_cast<const uint32_t*>(row_base) + (bit >> 5);
    w[0] = __funnelshift_r(p[0], p[1], bit & 31);
  } else if constexpr (B == 4) {
    w[0] = *reinterpret_cast<const uint16_t*>(row_base + 2 * lane);
  } else if constexpr (B == 8) {
    w[0] = *reinterpret_cast<const uint32_t*>(row_base + 4 * lane);
  } else {
    const uint2 v = *reinterpret_cast<const uint2*>(row_base + 8 * lane);
    w[0] = v.x;
    w[1] = v.y;
  }
}

// code k of the lane as the float 2^23 + code (bit pattern 0x4B000000 | code)
template <int B>
__device__ __forceinline__ float code_as_float(const uint32_t (&w)[2], int k) {
  if constexpr (B == 8) {
    return __uint_as_float(__byte_perm(w[0], kTwo23Bits, 0x7440 | k));
  } else if constexpr (B == 16) {
    return __uint_as_float(__byte_perm(w[k >> 1], kTwo23Bits, (k & 1) ? 0x7432 : 0x7410));
  } else {
    return __uint_as_float(((w[0] >> (B * k)) & Wd<B>::mask) | kTwo23Bits);
  }
}

template <int B>
__device__ __forceinline__ void decode_lin_row(const uint32_t (&w)[2], float s, float (&out)[4]) {
  constexpr float invq = 1.0f / (float)Wd<B>::qmax;
  constexpr float off = kTwo23 + (float)Wd<B>::half;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float q = __fadd_rn(code_as_float<B>(w, k), -off);
    out[k] = __fmul_rn(s, __fmul_rn(q, invq));
  }
}

template <int B>
__device__ __forceinline__ void decode_log_row(const uint32_t (&w)[2], float s, const float* lut8, float (&out)[4]) {
  if constexpr (B == 8) {
#pragma unroll
    for (int k = 0; k < 4; ++k) out[k] = __fmul_rn(s, lut8[(w[0] >> (8 * k)) & 255u]);
  } else if constexpr (B <= 4) {
    // 2^(code - K): the code drops into the low bits of the exponent field (127 - K has them clear)
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t e = ((w[0] << (23 - B * k)) & (Wd<B>::mask << 23)) | (Wd<B>::emin << 23);
      out[k] = __fmul_rn(s, __uint_as_float(e));
    }
  } else {
    constexpr float cb = (float)Wd<B>::Roct / (float)Wd<B>::K;
    constexpr float off = kTwo23 + (float)Wd<B>::K;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float rf = __fadd_rn(code_as_float<B>(w, k), -off);
      out[k] = __fmul_rn(s, ex2_poly(__fmul_rn(rf, cb)));
    }
  }
}

// ---- variant of the log code with the piecewise-linear logarithm (widths 8 and 16), all integers ----
// Distances are differences of fp32 bit patterns (2^23 units per octave); a block covers 30 octaves.
template <int B>
struct Pl {
  static constexpr uint32_t A = B == 8 ? 4352u : 1118464u;               // 2^32 * K / (30 * 2^23), a whole number
  static constexpr uint32_t step = B == 8 ? 4042322161u : 4026593281u;   // round(30 * 2^23 * 2^S / K)
  static constexpr int S = B == 8 ? 12 : 20;
};
constexpr uint32_t kPlOctaves = 30u << 23;

// distance below the block maximum of the level j code steps below it: floor(j * step / 2^S + 1/2)
template <int B>
__device__ __forceinline__ uint32_t pl_below(uint32_t j) {
  return (uint32_t)(((unsigned long long)j * Pl<B>::step + (1ull << (Pl<B>::S - 1))) >> Pl<B>::S);
}
__device__ __forceinline__ float pl_value(uint32_t s_bits, uint32_t below) {
  return __uint_as_float((uint32_t)max((int)s_bits - (int)below, 0));
}

// lutn: pl_below<8>(j) for j = 0..255
template <int B>
__device__ __forceinline__ void decode_pl_row(const uint32_t (&w)[2], uint32_t s_bits, const uint32_t* lutn,
                                              float (&out)[4]) {
  if constexpr (B == 8) {
    const uint32_t nw = ~w[0];          // K - code per field
#pragma unroll
    for (int k = 0; k < 4; ++k) out[k] = pl_value(s_bits, lutn[(nw >> (8 * k)) & 255u]);
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t nw = ~w[k >> 1];
      out[k] = pl_value(s_bits, pl_below<16>((k & 1) ? nw >> 16 : nw & 0xFFFFu));
    }
  }
}

// Stores the lane's packed field(s) of one row.  f: the 4*B-bit field (two words at 16 bits).
template <int B>
__device__ __forceinline__ void store_fields(uint8_t* row_ptr, int lane, uint32_t f0, uint32_t f1) {
  if constexpr (B == 2) {
    *(row_ptr + lane) = (uint8_t)f0;
  } else if constexpr (B == 3) {
    // a lane pair shares three bytes: even lane owns bits 0..11, odd lane bits 12..23
    const uint32_t p = f0 & 0xFFFu;
    const uint32_t other = __shfl_xor_sync(kFull, p, 1);
    uint8_t* base = row_ptr + 3 * (lane >> 1);
    const bool odd = lane & 1;
    *(base + (odd ? 2 : 0)) = (uint8_t)(odd ? (p >> 4) : p);
    if (!odd) *(base + 1) = (uint8_t)((p >> 8) | (other << 4));
  } else if constexpr (B == 4) {
    *reinterpret_cast<uint16_t*>(row_ptr + 2 * lane) = (uint16_t)f0;
  } else if constexpr (B == 8) {
    *reinterpret_cast<uint32_t*>(row_ptr + 4 * lane) = f0;
  } else {
    *reinterpret_cast<uint2*>(row_ptr + 8 * lane) = make_uint2(f0, f1);
  }
}

// Packs x_k = base + u_k (u_k < 2^B) and stores the row's codes.
template <int B>
__device__ __forceinline__ void pack_store_row(uint8_t* row_ptr, int lane, const uint32_t (&x)[4], uint32_t base) {
  if constexpr (B == 16) {
    store_fields<B>(row_ptr, lane, x[0] + (x[1] << 16) - base * Wd<16>::fieldsum,
                    x[2] + (x[3] << 16) - base * Wd<16>::fieldsum);
  } else {
    store_fields<B>(row_ptr, lane, x[0] + (x[1] << B) + (x[2] << (2 * B)) + (x[3] << (3 * B)) - base * Wd<B>::fieldsum, 0u);
  }
}

// Quantize one row of new first moments and store the codes.  mq receives what the update needs:
// the decoded values times `gain` = lr/(1-beta1^t), formed as q * (s * gain / qmax) (the update is
// held to 1e-6, not to the bit, so the two roundings of the decode are merged into one factor).
template <int B>
__device__ __forceinline__ void encode_lin_row(uint8_t* row_ptr, int lane, const float (&m)[4], float s_gain, float inv,
                                               float (&mq)[4]) {
  constexpr float invq = 1.0f / (float)Wd<B>::qmax;
  constexpr float mg = kMagic + (float)Wd<B>::half;
  const float unit = __fmul_rn(s_gain, invq);
  uint32_t x[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float t = __fmaf_rn(m[k], inv, mg);
    x[k] = __float_as_uint(t);
    mq[k] = __fmul_rn(__fadd_rn(t, -mg), unit);
  }
  pack_store_row<B>(row_ptr, lane, x, kMagicBits);
}

// Quantize one row of new second moments.  lgc: sqrt2/s (octave widths) or P(s) (8, 16 bits);
// ebase: kMagicBits - E_s (8, 16 bits).
template <int B>
__device__ __forceinline__ void encode_log_row(uint8_t* row_ptr, int lane, const float (&v)[4], float s, float lgc,
                                               uint32_t ebase, const float* lut8, float (&vq)[4]) {
  if constexpr (B <= 4) {
    const float ymin = __uint_as_float(Wd<B>::emin << 23);
    uint32_t f = 0u;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      // exponent of x*sqrt2/s, floored at -K: its low B bits are the code
      const uint32_t yb = __float_as_uint(fmaxf(__fmul_rn(v[k], lgc), ymin));
      f |= (yb >> (23 - B * k)) & (Wd<B>::mask << (B * k));
      vq[k] = __fmul_rn(s, __uint_as_float(yb & 0x7F800000u));
    }
    store_fields<B>(row_ptr, lane, f, 0u);
  } else {
    constexpr float a = (float)Wd<B>::K / (float)Wd<B>::Roct;
    constexpr float cb = (float)Wd<B>::Roct / (float)Wd<B>::K;
    constexpr float negR = -(float)Wd<B>::Roct;
    uint32_t x[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t xb = __float_as_uint(v[k]);
      const float de = __fadd_rn(__uint_as_float(ebase + (xb >> 23)), -kMagic);
      const float dp = __fadd_rn(lg_poly(xb), -lgc);
      const float d = fmaxf(__fadd_rn(de, dp), negR);
      const float t = __fmaf_rn(d, a, kMagic);
      x[k] = __float_as_uint(t);
      if constexpr (B == 8) vq[k] = __fmul_rn(s, lut8[(x[k] + 255u) & 255u]);   // low bits are code - 255
      else vq[k] = __fmul_rn(s, ex2_poly(__fmul_rn(__fadd_rn(t, -kMagic), cb)));
    }
    pack_store_row<B>(row_ptr, lane, x, kMagicBits - (uint32_t)Wd<B>::K);
  }
}

// The same in the piecewise-linear variant.  s_enc: bit pattern of the block maximum (+inf's for a
// zero block, which floors every code); s_dec: the same, 0 for a zero block.
template <int B>
__device__ __forceinline__ void encode_pl_row(uint8_t* row_ptr, int lane, const float (&v)[4], uint32_t s_enc,
                                              uint32_t s_dec, const uint32_t* lutn, float (&vq)[4]) {
  uint32_t j[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t n = min(s_enc - __float_as_uint(v[k]), kPlOctaves);
    j[k] = (uint32_t)(((unsigned long long)n * Pl<B>::A + (1ull << 31)) >> 32);   // floor(n*K/D + 1/2) <= K
    uint32_t below;
    if constexpr (B == 8) below = lutn[j[k]];
    else below = pl_below<16>(j[k]);
    vq[k] = pl_value(s_dec, below);
  }
  // code = K - j: the complement of j inside its field
  if constexpr (B == 8) store_fields<8>(row_ptr, lane, ~(j[0] | (j[1] << 8) | (j[2] << 16) | (j[3] << 24)), 0u);
  else store_fields<16>(row_ptr, lane, ~(j[0] | (j[1] << 16)), ~(j[2] | (j[3] << 16)));
}

__device__ __forceinline__ float ex2_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- the update's share of the fused bodies ----------------------------------------------------------
// The parameter update is held to 1e-6, not to the bit, so the fused bodies do not decode the new codes
// again: they take what the update needs straight from the encode.
//
// First moment: q = code - 2^(B-1) as a float (the caller multiplies by scale * lr/(1-beta1^t) / qmax).
template <int B>
__device__ __forceinline__ void encode_lin_row_q(uint8_t* row_ptr, int lane, const float (&m)[4], float inv,
                                                 float (&q)[4]) {
  constexpr float mg = kMagic + (float)Wd<B>::half;
  uint32_t x[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float t = __fmaf_rn(m[k], inv, mg);
    x[k] = __float_as_uint(t);
    q[k] = __fadd_rn(t, -mg);
  }
  pack_store_row<B>(row_ptr, lane, x, kMagicBits);
}

// Octave code (B <= 4) of one row of new second moments.  A block has only 2^B levels, so the factor
// every level contributes to the update is worked out once per row by 2^B lanes (tile_body) and fetched
// with a shuffle.  The shuffle takes its source lane from the low five bits of its operand, so the
// products are scaled by a power of two chosen per row (c_up = sqrt2/s * 2^u, ymin_up = 2^(u-K)) such
// that the exponent field of y itself ends in (row's first lane + code): e[k] is that operand.  u is a
// multiple of 2^B, so the code (the low B bits of the exponent) is what it was; scaling up cannot
// overflow (c <= sqrt2 * 2^100, u <= 16) and is exact, and whatever underflows is below the floor
// level in either scaling.
template <int B>
struct Oct {
  static constexpr int NL = 1 << B;
  static constexpr int up0 = (64 - (int)(Wd<B>::emin & 31u)) & 31;        // first row of the pass: lanes 0 .. NL-1
  static constexpr int up1 = (NL + 64 - (int)(Wd<B>::emin & 31u)) & 31;   // second row: lanes NL .. 2 NL-1
};
template <int B>
__device__ __forceinline__ void encode_oct_row(uint8_t* row_ptr, int lane, const float (&v)[4], float c_up,
                                               float ymin_up, uint32_t (&e)[4]) {
  uint32_t f = 0u;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t yb = __float_as_uint(fmaxf(__fmul_rn(v[k], c_up), ymin_up));
    f |= (yb >> (23 - B * k)) & (Wd<B>::mask << (B * k));
    e[k] = yb >> 23;
  }
  store_fields<B>(row_ptr, lane, f, 0u);
}

// Polynomial log code (B = 8, 16): r = code - K as a float (the update forms 2^(r * R/K / 2) itself).
template <int B>
__device__ __forceinline__ void encode_log_row_r(uint8_t* row_ptr, int lane, const float (&v)[4], float lgc,
                                                 uint32_t ebase, float (&r)[4]) {
  constexpr float a = (float)Wd<B>::K / (float)Wd<B>::Roct;
  constexpr float negR = -(float)Wd<B>::Roct;
  uint32_t x[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t xb = __float_as_uint(v[k]);
    const float de = __fadd_rn(__uint_as_float(ebase + (xb >> 23)), -kMagic);
    const float dp = __fadd_rn(lg_poly(xb), -lgc);
    const float d = fmaxf(__fadd_rn(de, dp), negR);
    const float t = __fmaf_rn(d, a, kMagic);
    x[k] = __float_as_uint(t);
    r[k] = __fadd_rn(t, -kMagic);
  }
  pack_store_row<B>(row_ptr, lane, x, kMagicBits - (uint32_t)Wd<B>::K);
}

template <int GDT>
__device__ __forceinline__ void lds_grad(const uint8_t* stage, int elem, float (&g)[4]) {
  if constexpr (GDT == 0) {
    const float4 v = *reinterpret_cast<const float4*>(stage + kOffGrad + 4 * elem);
    g[0] = v.x; g[1] = v.y; g[2] = v.z; g[3] = v.w;
  } else if constexpr (GDT == 1) {
    const uint2 v = *reinterpret_cast<const uint2*>(stage + kOffGrad + 2 * elem);
    g[0] = __uint_as_float(v.x << 16);
    g[1] = __uint_as_float(v.x & 0xFFFF0000u);
    g[2] = __uint_as_float(v.y << 16);
    g[3] = __uint_as_float(v.y & 0xFFFF0000u);
  } else {
    const uint2 v = *reinterpret_cast<const uint2*>(stage + kOffGrad + 2 * elem);
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
    g[0] = a.x; g[1] = a.y; g[2] = b.x; g[3] = b.y;
  }
}

// Four updated parameters rounded (nearest-even) to the working precision of the model.
__device__ __forceinline__ uint2 pack_lp(const float (&x)[4], uint32_t lp_dtype) {
  uint2 r;
  if (lp_dtype == 1u) {
    const __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]), b = __floats2bfloat162_rn(x[2], x[3]);
    r.x = *reinterpret_cast<const uint32_t*>(&a);
    r.y = *reinterpret_cast<const uint32_t*>(&b);
  } else {
    const __half2 a = __floats2half2_rn(x[0], x[1]), b = __floats2half2_rn(x[2], x[3]);
    r.x = *reinterpret_cast<const uint32_t*>(&a);
    r.y = *reinterpret_cast<const uint32_t*>(&b);
  }
  return r;
}

// ---- two elements per instruction ----------------------------------------------------------------------
// sm_100 executes fp32 add, multiply and fused multiply-add on register pairs (two independent IEEE
// operations per instruction, each rounded exactly as the scalar one).  The step is bound by instruction
// issue as much as by memory, and a third of its instructions are fp32 arithmetic on a lane's four
// elements, so the fused bodies keep those as two pairs and do the per-element arithmetic pairwise
// (PTX add / mul / fma .rn.f32x2 through the toolkit's intrinsics).
// One trap: the assembler contracts a packed multiply whose only use is a packed add into one packed fused
// multiply-add, explicit rounding modifiers and -fmad=false notwithstanding (measured: 0.35 % of random
// operands change).  The quantizers are defined with separate roundings, so wherever a packed product
// meets a sum the sum is written as fma(x, one, y) with `one` = 1.0f that the assembler cannot know (a
// launch parameter): the same value as x + y, and nothing to contract.
using f2 = float2;
__device__ __forceinline__ f2 splat(float x) { return make_float2(x, x); }
__device__ __forceinline__ f2 add2(f2 a, f2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ f2 mul2(f2 a, f2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ f2 fma2(f2 a, f2 b, f2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ f2 bits2(uint32_t a, uint32_t b) { return make_float2(__uint_as_float(a), __uint_as_float(b)); }

template <int B>
__device__ __forceinline__ f2 code_pair(const uint32_t (&w)[2], int h) {
  return make_float2(code_as_float<B>(w, 2 * h), code_as_float<B>(w, 2 * h + 1));
}

template <int B>
__device__ __forceinline__ void decode_lin_pairs(const uint32_t (&w)[2], float s, f2 (&out)[2]) {
  constexpr float invq = 1.0f / (float)Wd<B>::qmax;
  constexpr float off = kTwo23 + (float)Wd<B>::half;
  const f2 s2 = splat(s);
#pragma unroll
  for (int h = 0; h < 2; ++h) out[h] = mul2(s2, mul2(add2(code_pair<B>(w, h), splat(-off)), splat(invq)));
}

// 2^e (e <= 0) of a pair, the same operations as ex2_poly (e is a product: its sum goes through `one`)
__device__ __forceinline__ f2 ex2_poly_pair(f2 e, f2 one) {
  const f2 ti = fma2(e, one, splat(kMagic));
  const f2 fi = add2(ti, splat(-kMagic));
  const f2 f = fma2(fi, splat(-1.0f), e);          // e - fi, exact
  f2 a = splat(kE4);
  a = fma2(a, f, splat(kE3));
  a = fma2(a, f, splat(kE2));
  a = fma2(a, f, splat(kE1));
  a = fma2(a, f, splat(kE0));
  const f2 p = fma2(a, f, splat(1.0f));
  return bits2(__float_as_uint(p.x) + (__float_as_uint(ti.x) << 23), __float_as_uint(p.y) + (__float_as_uint(ti.y) << 23));
}
// P(mantissa) of a pair of bit patterns, the same operations as lg_poly
__device__ __forceinline__ f2 lg_poly_pair(uint32_t b0, uint32_t b1) {
  const f2 mant = bits2((b0 & 0x007FFFFFu) | 0x3F800000u, (b1 & 0x007FFFFFu) | 0x3F800000u);
  const f2 t = add2(mant, splat(-1.0f));
  f2 a = splat(kP6);
  a = fma2(a, t, splat(kP5));
  a = fma2(a, t, splat(kP4));
  a = fma2(a, t, splat(kP3));
  a = fma2(a, t, splat(kP2));
  a = fma2(a, t, splat(kP1));
  return mul2(a, t);
}

template <int B>
__device__ __forceinline__ void decode_log_pairs(const uint32_t (&w)[2], float s, const float* lut8, f2 one,
                                                 f2 (&out)[2]) {
  const f2 s2 = splat(s);
  if constexpr (B == 8) {
#pragma unroll
    for (int h = 0; h < 2; ++h)
      out[h] = mul2(s2, make_float2(lut8[(w[0] >> (16 * h)) & 255u], lut8[(w[0] >> (16 * h + 8)) & 255u]));
  } else if constexpr (B <= 4) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t e0 = ((w[0] << (23 - B * (2 * h))) & (Wd<B>::mask << 23)) | (Wd<B>::emin << 23);
      const uint32_t e1 = ((w[0] << (23 - B * (2 * h + 1))) & (Wd<B>::mask << 23)) | (Wd<B>::emin << 23);
      out[h] = mul2(s2, bits2(e0, e1));
    }
  } else {
    constexpr float cb = (float)Wd<B>::Roct / (float)Wd<B>::K;
    constexpr float off = kTwo23 + (float)Wd<B>::K;
#pragma unroll
    for (int h = 0; h < 2; ++h)
      out[h] = mul2(s2, ex2_poly_pair(mul2(add2(code_pair<B>(w, h), splat(-off)), splat(cb)), one));
  }
}

// Quantize one row of new first moments and store the codes; nq = 2^(B-1) - code = -q as floats.
template <int B>
__device__ __forceinline__ void encode_lin_pairs(uint8_t* row_ptr, int lane, const f2 (&m)[2], float inv, f2 (&nq)[2]) {
  constexpr float mg = kMagic + (float)Wd<B>::half;
  uint32_t x[4];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const f2 t = fma2(m[h], splat(inv), splat(mg));
    x[2 * h] = __float_as_uint(t.x);
    x[2 * h + 1] = __float_as_uint(t.y);
    nq[h] = fma2(t, splat(-1.0f), splat(mg));       // mg - t, exact
  }
  pack_store_row<B>(row_ptr, lane, x, kMagicBits);
}

// Octave code of one row of new second moments (see encode_oct_row): codes stored, e = exponent fields.
template <int B>
__device__ __forceinline__ void encode_oct_pairs(uint8_t* row_ptr, int lane, const f2 (&v)[2], float c_up, float ymin_up,
                                                 uint32_t (&e)[4]) {
  uint32_t f = 0u;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const f2 y = mul2(v[h], splat(c_up));
    const uint32_t y0 = __float_as_uint(fmaxf(y.x, ymin_up)), y1 = __float_as_uint(fmaxf(y.y, ymin_up));
    f |= (y0 >> (23 - B * (2 * h))) & (Wd<B>::mask << (B * (2 * h)));
    f |= (y1 >> (23 - B * (2 * h + 1))) & (Wd<B>::mask << (B * (2 * h + 1)));
    e[2 * h] = y0 >> 23;
    e[2 * h + 1] = y1 >> 23;
  }
  store_fields<B>(row_ptr, lane, f, 0u);
}

// Polynomial log code (8, 16 bits) of one row; r = code - K as floats.
template <int B>
__device__ __forceinline__ void encode_log_pairs(uint8_t* row_ptr, int lane, const f2 (&v)[2], float lgc, uint32_t ebase,
                                                 f2 one, f2 (&r)[2]) {
  constexpr float a = (float)Wd<B>::K / (float)Wd<B>::Roct;
  constexpr float negR = -(float)Wd<B>::Roct;
  uint32_t x[4];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const uint32_t b0 = __float_as_uint(v[h].x), b1 = __float_as_uint(v[h].y);
    const f2 de = add2(bits2(ebase + (b0 >> 23), ebase + (b1 >> 23)), splat(-kMagic));
    const f2 dp = fma2(lg_poly_pair(b0, b1), one, splat(-lgc));      // P(x) - P(s): a product meets a sum
    f2 d = add2(de, dp);
    d = make_float2(fmaxf(d.x, negR), fmaxf(d.y, negR));
    const f2 t = fma2(d, splat(a), splat(kMagic));
    x[2 * h] = __float_as_uint(t.x);
    x[2 * h + 1] = __float_as_uint(t.y);
    r[h] = add2(t, splat(-kMagic));
  }
  pack_store_row<B>(row_ptr, lane, x, kMagicBits - (uint32_t)Wd<B>::K);
}

// One staged tile, one warp: R rows of 128 elements, taken in passes of RP rows.  The pass loop is
// a real loop (not unrolled): the straight-line body of a pass is what the warps stream through the
// instruction cache, and halving it pays more than the lost overlap between passes.  Specialised on
// both widths.
constexpr int RP = kFastRowsPerPass;
template <int BM, int BV, bool VPL, int GDT, bool AMP>
__device__ __forceinline__ void tile_body(const uint8_t* __restrict__ stage, const TileInfo& ti, const StepConsts& sc,
                                          const float* __restrict__ lut8, int lane, int warp, uint32_t empty_bar,
                                          double* __restrict__ part, float grad_mul) {
  static_assert(!VPL || BV >= 8, "the piecewise-linear variant exists at 8 and 16 bits");
  static_assert(RP == 2, "the level shuffle of the octave codes is laid out for two rows per pass");
  [[maybe_unused]] const uint32_t* lutn = reinterpret_cast<const uint32_t*>(lut8 + 256);
  const int lgB = (int)((ti.packed >> 16) & 0xFFu);
  [[maybe_unused]] const uint32_t lp_dtype = ti.packed >> 24;
  const float nlrwd = sc.l2_mode ? 0.0f : -ti.wdx;
  f2 a0 = splat(0.f), a1 = splat(0.f), a2 = splat(0.f);      // statistics over the raw gradient (decision steps)
  const f2 one2 = splat(sc.one);
  // octave v codes: 2^(level - K) of the level this lane tabulates for the update (see below)
  constexpr int LV = BV <= 4 ? BV : 2;
  [[maybe_unused]] const float lvl = __uint_as_float((((uint32_t)lane & Wd<LV>::mask) + Wd<LV>::emin) << 23);

#pragma unroll 1
  for (int pass = 0; pass < R / RP; ++pass) {
    const int row0 = warp * R + pass * RP;

    // ---- staged rows -> registers, decode -----------------------------------------------------------
    f2 th[RP][2], g[RP][2], mt[RP][2], vt[RP][2];
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      const int elem = (row0 + r) * kRowElems + 4 * lane;
      const float4 t4 = *reinterpret_cast<const float4*>(stage + kOffTheta + 4 * elem);
      th[r][0] = make_float2(t4.x, t4.y);
      th[r][1] = make_float2(t4.z, t4.w);
      float gs[4];
      lds_grad<GDT>(stage, elem, gs);
      g[r][0] = make_float2(gs[0], gs[1]);
      g[r][1] = make_float2(gs[2], gs[3]);
      const int blk = ((row0 + r) * kRowElems) >> lgB;
      const float sm = *reinterpret_cast<const float*>(stage + kOffMs + 4 * blk);
      const float sv = *reinterpret_cast<const float*>(stage + kOffVs + 4 * blk);
      uint32_t w[2];
      lds_codes<BM>(stage + kOffMc + (row0 + r) * (16 * BM), lane, w);
      decode_lin_pairs<BM>(w, sm, mt[r]);
      lds_codes<BV>(stage + kOffVc + (row0 + r) * (16 * BV), lane, w);
      if constexpr (VPL) {
        float vs[4];
        decode_pl_row<BV>(w, __float_as_uint(sv), lutn, vs);
        vt[r][0] = make_float2(vs[0], vs[1]);
        vt[r][1] = make_float2(vs[2], vs[3]);
      } else {
        decode_log_pairs<BV>(w, sv, lut8, one2, vt[r]);
      }
    }
    if (pass == R / RP - 1) {   // the last rows are in registers: this warp is done with the stage
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar);
    }

    if constexpr (AMP) {               // loss-scaled gradients: back to true scale first (x1 is exact)
#pragma unroll
      for (int r = 0; r < RP; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) g[r][h] = mul2(g[r][h], splat(grad_mul));
    }
    if (part != nullptr) {
#pragma unroll
      for (int r = 0; r < RP; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          a0 = fma2(g[r][h], one2, a0);       // (g may be a product: the unscaled gradient)
          a1 = add2(a1, make_float2(fabsf(g[r][h].x), fabsf(g[r][h].y)));
          a2 = fma2(g[r][h], g[r][h], a2);
        }
    }

    // ---- moments ----------------------------------------------------------------------------------------
    if (sc.l2_mode) {
#pragma unroll
      for (int r = 0; r < RP; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) g[r][h] = fma2(g[r][h], one2, mul2(splat(ti.wdx), th[r][h]));
    }
#pragma unroll
    for (int r = 0; r < RP; ++r) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const f2 gk = g[r][h];
        mt[r][h] = fma2(splat(sc.b1), mt[r][h], mul2(splat(sc.c1), gk));
        vt[r][h] = fma2(splat(sc.b2), vt[r][h], mul2(mul2(splat(sc.c2), gk), gk));
      }
    }

    // ---- block maxima --------------------------------------------------------------------------------
    uint32_t mxm[RP], mxv[RP];
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      const float am = fmaxf(fmaxf(fabsf(mt[r][0].x), fabsf(mt[r][0].y)), fmaxf(fabsf(mt[r][1].x), fabsf(mt[r][1].y)));
      const float av = fmaxf(fmaxf(vt[r][0].x, vt[r][0].y), fmaxf(vt[r][1].x, vt[r][1].y));
      mxm[r] = __reduce_max_sync(kFull, __float_as_uint(am));
      mxv[r] = __reduce_max_sync(kFull, __float_as_uint(av));
    }
    if (lgB >= 8) {
      mxm[0] = mxm[1] = max(mxm[0], mxm[1]);
      mxv[0] = mxv[1] = max(mxv[0], mxv[1]);
    }

    // ---- per-block constants: one lane per (row, state) works them out, then they are broadcast --------
    // lanes 0..RP-1: inv = fl(qmax * fl(1/s_m));  lanes RP..2RP-1 (octave widths): c = fl(sqrt2 * fl(1/s_v)),
    // times the power of two that steers the level shuffle of its row (encode_oct_row)
    float inv_m[RP], lgc[RP];
    {
      uint32_t mine = (lane & 1) ? mxm[1] : mxm[0];
      if constexpr (BV <= 4) {
        if (lane & RP) mine = (lane & 1) ? mxv[1] : mxv[0];
      }
      const float x = __uint_as_float(mine);
      const bool zero = x < kTiny;
      float mul = (float)Wd<BM>::qmax;
      if constexpr (BV <= 4) {
        constexpr float up0 = kSqrt2 * (float)(1 << Oct<LV>::up0);
        constexpr float up1 = kSqrt2 * (float)(1 << Oct<LV>::up1);
        if (lane & RP) mul = (lane & 1) ? up1 : up0;
      }
      const float val = zero ? 0.f : __fmul_rn(mul, __frcp_rn(x));
      // the same lanes store the new scales (a zero block stores 0), for the rows that open a block
      const int e_mine = (row0 + (lane & (RP - 1))) * kRowElems;
      const bool opens = (e_mine & ((1 << lgB) - 1)) == 0;
#pragma unroll
      for (int r = 0; r < RP; ++r) inv_m[r] = __shfl_sync(kFull, val, r);
      if constexpr (BV <= 4) {
        if (lane < 2 * RP && opens) ((lane & RP) ? ti.vso : ti.mso)[e_mine >> lgB] = zero ? 0.f : x;
#pragma unroll
        for (int r = 0; r < RP; ++r) lgc[r] = __shfl_sync(kFull, val, RP + r);
      } else {
        const uint32_t mv = (lane & 1) ? mxv[1] : mxv[0];
        if (lane < RP && opens) {
          ti.mso[e_mine >> lgB] = zero ? 0.f : x;
          ti.vso[e_mine >> lgB] = __uint_as_float(mv) < kTiny ? 0.f : __uint_as_float(mv);
        }
        if constexpr (!VPL) {
          const float ps = lg_poly(mv);
#pragma unroll
          for (int r = 0; r < RP; ++r) lgc[r] = __shfl_sync(kFull, ps, r);
        } else {
#pragma unroll
          for (int r = 0; r < RP; ++r) lgc[r] = 0.f;
        }
      }
    }

    // ---- octave v codes: what each level of each row contributes to the update, one level per lane -----
    // lane l: level (l mod 2^BV) of row (l div 2^BV) of the pass; value lr/(1-beta1^t) * s_m/qmax /
    // (sqrt(s_v * 2^(level-K) / (1-beta2^t)) + eps), so that the update of an element is q_m times the
    // entry of its level.  (An all-zero block of v has s_v = 0: every level gives 1/eps, as its decode would.)
    [[maybe_unused]] float lut_upd = 0.f;
    if constexpr (BV <= 4) {
      constexpr float invq = 1.0f / (float)Wd<BM>::qmax;
      const bool second = (lane >> LV) & 1;
      const float svr = __uint_as_float(second ? mxv[1] : mxv[0]);
      const float smr = __uint_as_float(second ? mxm[1] : mxm[0]);
      const float vl = __fmul_rn(svr < kTiny ? 0.f : svr, lvl);
      const float den = __fmaf_rn(sqrt_fast(vl), sc.rsqrt_bc2, sc.eps);
      lut_upd = __fmul_rn(__fmul_rn(__fmul_rn(smr, sc.step_size), invq), rcp_fast(den));
    }

    // ---- quantize, pack, store; update the parameters ---------------------------------------------------
    // theta - lr*wd*theta - update as fma(-q, factor, fma(theta, -lr*wd, theta)): the decay keeps its own
    // precision (a factor 1 - lr*wd rounded to fp32 would be off by ~1e-3 of the decay it applies)
    float* param = ti.param + row0 * kRowElems + 4 * lane;
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      // A zero block of m needs no special case here: its inv is 0, so every q is 0 and so is the update.
      const float sm_raw = __uint_as_float(mxm[r]);
      const float sv_raw = __uint_as_float(mxv[r]);
      const bool vzero = sv_raw < kTiny;
      f2 out[2];
      if constexpr (BV <= 4) {
        f2 nq[2];
        uint32_t e[4];
        encode_lin_pairs<BM>(ti.mco + (row0 + r) * (16 * BM), lane, mt[r], inv_m[r], nq);
        const float ymin_up = __uint_as_float((Wd<LV>::emin + (uint32_t)(r == 0 ? Oct<LV>::up0 : Oct<LV>::up1)) << 23);
        encode_oct_pairs<LV>(ti.vco + (row0 + r) * (16 * BV), lane, vt[r], lgc[r], ymin_up, e);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const f2 base = fma2(th[r][h], splat(nlrwd), th[r][h]);
          const f2 fac = make_float2(__shfl_sync(kFull, lut_upd, e[2 * h]), __shfl_sync(kFull, lut_upd, e[2 * h + 1]));
          out[h] = fma2(nq[h], fac, base);
        }
      } else if constexpr (!VPL) {
        // 2^((code-K) * R/K / 2) by the special-function unit: sqrt of the decoded level, to 2^-22
        constexpr int LB = BV >= 8 ? BV : 8;
        constexpr float half_cb = 0.5f * ((float)Wd<LB>::Roct / (float)Wd<LB>::K);
        constexpr float invq = 1.0f / (float)Wd<BM>::qmax;
        const uint32_t ebase = kMagicBits - (vzero ? (uint32_t)kZeroBlockExp : (mxv[r] >> 23));
        const float unit = __fmul_rn(__fmul_rn(sm_raw, sc.step_size), invq);
        const float srt = __fmul_rn(sqrt_fast(vzero ? 0.f : sv_raw), sc.rsqrt_bc2);
        f2 nq[2], rr[2];
        encode_lin_pairs<BM>(ti.mco + (row0 + r) * (16 * BM), lane, mt[r], inv_m[r], nq);
        encode_log_pairs<LB>(ti.vco + (row0 + r) * (16 * BV), lane, vt[r], lgc[r], ebase, one2, rr);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const f2 arg = mul2(rr[h], splat(half_cb));
          const f2 den = fma2(make_float2(ex2_fast(arg.x), ex2_fast(arg.y)), splat(srt), splat(sc.eps));
          const f2 base = fma2(th[r][h], splat(nlrwd), th[r][h]);
          out[h] = fma2(mul2(nq[h], splat(unit)), make_float2(rcp_fast(den.x), rcp_fast(den.y)), base);
        }
      } else {
        constexpr int LB = BV >= 8 ? BV : 8;
        constexpr float invq = 1.0f / (float)Wd<BM>::qmax;
        const float unit = __fmul_rn(__fmul_rn(sm_raw, sc.step_size), invq);
        f2 nq[2];
        float vs[4], vq[4];
        encode_lin_pairs<BM>(ti.mco + (row0 + r) * (16 * BM), lane, mt[r], inv_m[r], nq);
        vs[0] = vt[r][0].x; vs[1] = vt[r][0].y; vs[2] = vt[r][1].x; vs[3] = vt[r][1].y;
        encode_pl_row<LB>(ti.vco + (row0 + r) * (16 * BV), lane, vs, vzero ? 0x7F800000u : mxv[r],
                          vzero ? 0u : mxv[r], lutn, vq);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const f2 den = fma2(make_float2(sqrt_fast(vq[2 * h]), sqrt_fast(vq[2 * h + 1])), splat(sc.rsqrt_bc2), splat(sc.eps));
          const f2 base = fma2(th[r][h], splat(nlrwd), th[r][h]);
          out[h] = fma2(mul2(nq[h], splat(unit)), make_float2(rcp_fast(den.x), rcp_fast(den.y)), base);
        }
      }
      *reinterpret_cast<float4*>(param + r * kRowElems) = make_float4(out[0].x, out[0].y, out[1].x, out[1].y);
      if constexpr (AMP) {
        if (ti.lp != nullptr) {
          const float o4[4] = {out[0].x, out[0].y, out[1].x, out[1].y};
          *reinterpret_cast<uint2*>(ti.lp + (row0 + r) * kRowElems + 4 * lane) = pack_lp(o4, lp_dtype);
        }
      }
    }
  }

  if (part != nullptr) {
    // Pairwise fp32 butterfly that spreads the three sums over the lanes on the way down:
    // after xor 16 the low half carries (sum0, sum1) and the high half (sum2, -); after xor 8
    // lanes 0-7 / 8-15 / 16-23 carry sum0 / sum1 / sum2; three more steps finish each group.
    const float s0 = a0.x + a0.y, s1 = a1.x + a1.y, s2 = a2.x + a2.y;
    const bool hi = lane & 16;
    float x = (hi ? s2 : s0) + __shfl_xor_sync(kFull, hi ? s0 : s2, 16);
    float y = (hi ? 0.f : s1) + __shfl_xor_sync(kFull, hi ? s1 : 0.f, 16);
    const bool q = lane & 8;
    float z = (q ? y : x) + __shfl_xor_sync(kFull, q ? x : y, 8);
    z += __shfl_xor_sync(kFull, z, 4);
    z += __shfl_xor_sync(kFull, z, 2);
    z += __shfl_xor_sync(kFull, z, 1);
    if ((lane & 7) == 0 && lane < 24) part[lane >> 3] = (double)z;
  }
}

// ---- fused bodies of the "sr" and the "ts" code of the second moment ------------------------------------------
// (their own launch and work list; the first moment, the moments and the update are those of tile_body)
template <int B>
__device__ __forceinline__ uint32_t code_of(const uint32_t (&w)[2], int k) {
  if constexpr (B == 16) return (w[k >> 1] >> (16 * (k & 1))) & 0xFFFFu;
  else return (w[0] >> (B * k)) & Wd<B>::mask;
}
// "sr": levels per octave 2^g, spacing of the levels in units of the bit pattern 2^sh, bit pattern of level 0
template <int B>
struct Sr {
  static constexpr int g = B == 8 ? 3 : B == 16 ? 11 : 0;
  static constexpr int sh = 23 - g;
  static constexpr uint32_t floor_bits = 0x3F800000u - ((uint32_t)Wd<B>::K << sh);
};
constexpr float kOnePlus = 0x1.000008p+0f;      // 1 + 2^-21: lifts the block maximum to or just above 1

// "ts": what a block's two scales give: everything the decode or the encode of its elements needs
struct TsRow {
  float W, inv_or_step, Phi;     // range in octaves; K / W (encode) or W / K (decode); P(hi)
};
template <int B>
__device__ __forceinline__ TsRow ts_row(uint32_t hi_bits, uint32_t lo_bits, bool for_encode) {
  TsRow t;
  t.Phi = lg_poly(hi_bits);
  const float de = (float)((int)(lo_bits >> 23) - (int)(hi_bits >> 23));
  const float dp = __fadd_rn(lg_poly(lo_bits), -t.Phi);
  float W = -__fadd_rn(de, dp);
  W = W > 30.0f ? 30.0f : W;
  t.W = W > 0.0f ? W : 0.0f;
  if (for_encode) t.inv_or_step = t.W > 0.0f ? __fdiv_rn((float)Wd<B>::K, t.W) : 0.0f;
  else t.inv_or_step = __fdiv_rn(t.W, (float)Wd<B>::K);
  return t;
}

template <int BM, int BV, int VM, int GDT, bool AMP>
__device__ __forceinline__ void tile_body_var(const uint8_t* __restrict__ stage, const TileInfo& ti, const StepConsts& sc,
                                              int lane, int warp, uint32_t empty_bar, double* __restrict__ part,
                                              float grad_mul) {
  static_assert(VM == 2 || VM == 3, "2: stochastic rounding, 3: two scales per block");
  static_assert(RP == 2, "rows are taken two per pass");
  constexpr int K = Wd<BV>::K;
  constexpr bool kSr = VM == 2, kTs = VM == 3;
  const int lgB = (int)((ti.packed >> 16) & 0xFFu);
  [[maybe_unused]] const uint32_t lp_dtype = ti.packed >> 24;
  const float nlrwd = sc.l2_mode ? 0.0f : -ti.wdx;
  f2 a0 = splat(0.f), a1 = splat(0.f), a2 = splat(0.f);
  const f2 one2 = splat(sc.one);
  // "sr" at <= 4 bits: the levels are s * 2^(level - K), the update's factor per level comes from a lane table
  constexpr int LV = BV <= 4 ? BV : 2;
  [[maybe_unused]] const float lvl = __uint_as_float((((uint32_t)lane & Wd<LV>::mask) + Wd<LV>::emin) << 23);

#pragma unroll 1
  for (int pass = 0; pass < R / RP; ++pass) {
    const int row0 = warp * R + pass * RP;

    // ---- "ts": the stored {hi, lo} of the two rows' blocks give range and step; lanes of equal parity work
    // out the same row, lane r's copy is handed to everyone
    [[maybe_unused]] float step_in[RP] = {0.f, 0.f};
    // at <= 4 bits a block has at most 16 levels: lane (r << LV | q) works out level q of row r once, the elements
    // fetch theirs by shuffle (the same arithmetic as the per-element decode of the wider codes, hence the same bits)
    [[maybe_unused]] float lut_dec = 0.f;
    if constexpr (kTs && BV <= 4) {
      const int blk_l = ((row0 + ((lane >> LV) & 1)) * kRowElems) >> lgB;
      const float2 hl = *reinterpret_cast<const float2*>(stage + kOffVs + 8 * blk_l);
      const TsRow tr = ts_row<BV>(__float_as_uint(hl.x), __float_as_uint(hl.y), false);
      const int q = lane & (int)Wd<LV>::mask;
      const float val = __fmul_rn(hl.x, ex2_poly(__fmul_rn((float)(q - K), tr.inv_or_step)));
      lut_dec = q == 0 ? hl.y : val;          // code 0 is the stored minimum itself
    } else if constexpr (kTs) {
      const int blk_l = ((row0 + (lane & 1)) * kRowElems) >> lgB;
      const float2 hl = *reinterpret_cast<const float2*>(stage + kOffVs + 8 * blk_l);
      const TsRow tr = ts_row<BV>(__float_as_uint(hl.x), __float_as_uint(hl.y), false);
#pragma unroll
      for (int r = 0; r < RP; ++r) step_in[r] = __shfl_sync(kFull, tr.inv_or_step, r);
    }

    // ---- staged rows -> registers, decode -----------------------------------------------------------
    f2 th[RP][2], g[RP][2], mt[RP][2], vt[RP][2];
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      const int elem = (row0 + r) * kRowElems + 4 * lane;
      const float4 t4 = *reinterpret_cast<const float4*>(stage + kOffTheta + 4 * elem);
      th[r][0] = make_float2(t4.x, t4.y);
      th[r][1] = make_float2(t4.z, t4.w);
      float gs[4];
      lds_grad<GDT>(stage, elem, gs);
      g[r][0] = make_float2(gs[0], gs[1]);
      g[r][1] = make_float2(gs[2], gs[3]);
      const int blk = ((row0 + r) * kRowElems) >> lgB;
      const float sm = *reinterpret_cast<const float*>(stage + kOffMs + 4 * blk);
      uint32_t w[2];
      lds_codes<BM>(stage + kOffMc + (row0 + r) * (16 * BM), lane, w);
      decode_lin_pairs<BM>(w, sm, mt[r]);
      lds_codes<BV>(stage + kOffVc + (row0 + r) * (16 * BV), lane, w);
      if constexpr (kSr) {
        // level of code c: the float with bits(level 0) + (c << spacing), times the scale
        const f2 s2 = splat(*reinterpret_cast<const float*>(stage + kOffVs + 4 * blk));
#pragma unroll
        for (int h = 0; h < 2; ++h)
          vt[r][h] = mul2(s2, bits2(Sr<BV>::floor_bits + (code_of<BV>(w, 2 * h) << Sr<BV>::sh),
                                    Sr<BV>::floor_bits + (code_of<BV>(w, 2 * h + 1) << Sr<BV>::sh)));
      } else if constexpr (BV <= 4) {
#pragma unroll
        for (int h = 0; h < 2; ++h)
          vt[r][h] = make_float2(__shfl_sync(kFull, lut_dec, (int)(code_of<BV>(w, 2 * h) | (uint32_t)(r << LV))),
                                 __shfl_sync(kFull, lut_dec, (int)(code_of<BV>(w, 2 * h + 1) | (uint32_t)(r << LV))));
      } else {
        const float2 hl = *reinterpret_cast<const float2*>(stage + kOffVs + 8 * blk);
        constexpr float off = kTwo23 + (float)K;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const f2 rf = add2(bits2(code_of<BV>(w, 2 * h) | kTwo23Bits, code_of<BV>(w, 2 * h + 1) | kTwo23Bits), splat(-off));
          const f2 val = mul2(splat(hl.x), ex2_poly_pair(mul2(rf, splat(step_in[r])), one2));
          // code 0 is the stored minimum itself
          vt[r][h] = make_float2(rf.x == -(float)K ? hl.y : val.x, rf.y == -(float)K ? hl.y : val.y);
        }
      }
    }
    if (pass == R / RP - 1) {   // the last rows are in registers: this warp is done with the stage
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar);
    }

    if constexpr (AMP) {
#pragma unroll
      for (int r = 0; r < RP; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) g[r][h] = mul2(g[r][h], splat(grad_mul));
    }
    if (part != nullptr) {
#pragma unroll
      for (int r = 0; r < RP; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          a0 = fma2(g[r][h], one2, a0);
          a1 = add2(a1, make_float2(fabsf(g[r][h].x), fabsf(g[r][h].y)));
          a2 = fma2(g[r][h], g[r][h], a2);
        }
    }

    // ---- moments ----------------------------------------------------------------------------------------
    if (sc.l2_mode) {
#pragma unroll
      for (int r = 0; r < RP; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) g[r][h] = fma2(g[r][h], one2, mul2(splat(ti.wdx), th[r][h]));
    }
#pragma unroll
    for (int r = 0; r < RP; ++r) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const f2 gk = g[r][h];
        mt[r][h] = fma2(splat(sc.b1), mt[r][h], mul2(splat(sc.c1), gk));
        vt[r][h] = fma2(splat(sc.b2), vt[r][h], mul2(mul2(splat(sc.c2), gk), gk));
      }
    }

    // ---- block maxima (and, for "ts", minima) ---------------------------------------------------------------
    uint32_t mxm[RP], mxv[RP];
    [[maybe_unused]] uint32_t mnv[RP];
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      const float am = fmaxf(fmaxf(fabsf(mt[r][0].x), fabsf(mt[r][0].y)), fmaxf(fabsf(mt[r][1].x), fabsf(mt[r][1].y)));
      const float av = fmaxf(fmaxf(vt[r][0].x, vt[r][0].y), fmaxf(vt[r][1].x, vt[r][1].y));
      mxm[r] = __reduce_max_sync(kFull, __float_as_uint(am));
      mxv[r] = __reduce_max_sync(kFull, __float_as_uint(av));
      if constexpr (kTs) {
        const float an = fminf(fminf(vt[r][0].x, vt[r][0].y), fminf(vt[r][1].x, vt[r][1].y));
        mnv[r] = __reduce_min_sync(kFull, __float_as_uint(an));
      }
    }
    if (lgB >= 8) {
      mxm[0] = mxm[1] = max(mxm[0], mxm[1]);
      mxv[0] = mxv[1] = max(mxv[0], mxv[1]);
      if constexpr (kTs) mnv[0] = mnv[1] = min(mnv[0], mnv[1]);
    }

    // ---- per-block constants: one lane per (row, state) works them out, then they are broadcast --------
    // lanes 0, 1: inv = fl(qmax * fl(1/s_m)) of rows 0, 1; "sr": lanes 2, 3: c1 = fl(fl(1/s_v) * (1 + 2^-21));
    // "ts": lanes of equal parity work out the new range of their row, lane r's copy is handed to everyone.
    // The same lanes store the new scales, for the rows that open a block (a zero block stores 0).
    float inv_m[RP];
    [[maybe_unused]] float c1[RP], tsW[RP], tsInv[RP], tsPhi[RP], tsLo[RP], tsHalf[RP];
    {
      uint32_t mine = (lane & 1) ? mxm[1] : mxm[0];
      if constexpr (kSr) {
        if (lane & RP) mine = (lane & 1) ? mxv[1] : mxv[0];
      }
      const float x = __uint_as_float(mine);
      const bool zero = x < kTiny;
      const float mul = (kSr && (lane & RP)) ? kOnePlus : (float)Wd<BM>::qmax;
      const float val = zero ? 0.f : __fmul_rn(mul, __frcp_rn(x));
      const int e_mine = (row0 + (lane & (RP - 1))) * kRowElems;
      const bool opens = (e_mine & ((1 << lgB) - 1)) == 0;
#pragma unroll
      for (int r = 0; r < RP; ++r) inv_m[r] = __shfl_sync(kFull, val, r);
      if constexpr (kSr) {
        if (lane < 2 * RP && opens) ((lane & RP) ? ti.vso : ti.mso)[e_mine >> lgB] = zero ? 0.f : x;
#pragma unroll
        for (int r = 0; r < RP; ++r) c1[r] = __shfl_sync(kFull, val, RP + r);
      } else {
        const uint32_t hi_b = (lane & 1) ? mxv[1] : mxv[0];
        const bool vz = __uint_as_float(hi_b) < kTiny;
        // the minimum, raised to the floor 2^-30 below the maximum
        const float lo = fmaxf(__uint_as_float((lane & 1) ? mnv[1] : mnv[0]), __fmul_rn(__uint_as_float(hi_b), 0x1p-30f));
        TsRow tr = ts_row<BV>(hi_b, __float_as_uint(lo), true);
        // an all-zero block: every code is 0 (one step over a range of one octave, with every distance clamped to it)
        const float half_l = vz ? 0.f : __fmul_rn(0.5f, __fdiv_rn(tr.W, (float)K));     // half a code step, for the update
        if (vz) { tr.W = 1.0f; tr.inv_or_step = (float)K; tr.Phi = 0.0f; }
        if (lane < RP && opens) {
          ti.mso[e_mine >> lgB] = zero ? 0.f : x;
          *reinterpret_cast<float2*>(ti.vso + 2 * (e_mine >> lgB)) = vz ? make_float2(0.f, 0.f) : make_float2(__uint_as_float(hi_b), lo);
        }
#pragma unroll
        for (int r = 0; r < RP; ++r) {
          tsW[r] = __shfl_sync(kFull, tr.W, r);
          tsInv[r] = __shfl_sync(kFull, tr.inv_or_step, r);
          tsPhi[r] = __shfl_sync(kFull, tr.Phi, r);
          tsLo[r] = __shfl_sync(kFull, vz ? 0.f : lo, r);
          tsHalf[r] = __shfl_sync(kFull, half_l, r);
        }
      }
    }

    // ---- <= 4 bits: what each level of each row contributes to the update, one level per lane -------------
    [[maybe_unused]] float lut_upd = 0.f;
    if constexpr (kTs && BV <= 4) {
      // sqrt of level q of the new code: sqrt(hi) * 2^((q-K) * W/K / 2), or sqrt(lo) for q = 0
      constexpr float invq = 1.0f / (float)Wd<BM>::qmax;
      const bool second = (lane >> LV) & 1;
      const float svr = __uint_as_float(second ? mxv[1] : mxv[0]);
      const float smr = __uint_as_float(second ? mxm[1] : mxm[0]);
      const int q = lane & (int)Wd<LV>::mask;
      const float srt_hi = __fmul_rn(sqrt_fast(svr < kTiny ? 0.f : svr), sc.rsqrt_bc2);
      const float arg = __fmul_rn((float)(q - K), second ? tsHalf[1] : tsHalf[0]);
      float den = __fmaf_rn(ex2_fast(arg), srt_hi, sc.eps);
      if (q == 0) den = __fmaf_rn(sqrt_fast(second ? tsLo[1] : tsLo[0]), sc.rsqrt_bc2, sc.eps);
      lut_upd = __fmul_rn(__fmul_rn(__fmul_rn(smr, sc.step_size), invq), rcp_fast(den));
    }
    if constexpr (kSr && BV <= 4) {
      constexpr float invq = 1.0f / (float)Wd<BM>::qmax;
      const bool second = (lane >> LV) & 1;
      const float svr = __uint_as_float(second ? mxv[1] : mxv[0]);
      const float smr = __uint_as_float(second ? mxm[1] : mxm[0]);
      const float vl = __fmul_rn(svr < kTiny ? 0.f : svr, lvl);
      const float den = __fmaf_rn(sqrt_fast(vl), sc.rsqrt_bc2, sc.eps);
      lut_upd = __fmul_rn(__fmul_rn(__fmul_rn(smr, sc.step_size), invq), rcp_fast(den));
    }

    // ---- quantize, pack, store; update the parameters ---------------------------------------------------
    float* param = ti.param + row0 * kRowElems + 4 * lane;
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      constexpr float invq = 1.0f / (float)Wd<BM>::qmax;
      const float sm_raw = __uint_as_float(mxm[r]);
      const float sv_raw = __uint_as_float(mxv[r]);
      const bool vzero = sv_raw < kTiny;
      f2 nq[2], out[2];
      encode_lin_pairs<BM>(ti.mco + (row0 + r) * (16 * BM), lane, mt[r], inv_m[r], nq);
      [[maybe_unused]] const float unit = __fmul_rn(__fmul_rn(sm_raw, sc.step_size), invq);
      uint8_t* vrow = ti.vco + (row0 + r) * (16 * BV);
      if constexpr (kSr) {
        // y = fl(x * c1) clamped to [level 0, 1]; n = bits(1.0) - bits(y); j = ((n << (9+g)) + word) >> 32 level
        // steps below the maximum (at most K by the clamp), code K - j.  The element's word is
        // mix32(index ^ key); index = row's first + 4*lane + k, and the first xor-shift of the chain is shared
        // by the lane's four elements (k touches the two lowest bits only).
        const uint32_t base = (ti.e0 + (uint32_t)((row0 + r) * kRowElems + 4 * lane)) ^ ti.sr_key;
        const uint32_t base1 = base ^ (base >> 16);
        const float floor_y = __uint_as_float(Sr<BV>::floor_bits);
        uint32_t code[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const f2 y = mul2(vt[r][h], splat(c1[r]));
          const float yc[2] = {fminf(fmaxf(y.x, floor_y), 1.0f), fminf(fmaxf(y.y, floor_y), 1.0f)};
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const int k = 2 * h + q;
            uint32_t wd = (base1 ^ (uint32_t)k) * 0x85EBCA6Bu;
            wd ^= wd >> 13; wd *= 0xC2B2AE35u; wd ^= wd >> 16;
            const uint32_t n = 0x3F800000u - __float_as_uint(yc[q]);
            const uint32_t j = (uint32_t)((((unsigned long long)n << (9 + Sr<BV>::g)) + wd) >> 32);
            code[k] = (uint32_t)K - j;
          }
        }
        pack_store_row<BV>(vrow, lane, code, 0u);
        if constexpr (BV <= 4) {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const f2 base_t = fma2(th[r][h], splat(nlrwd), th[r][h]);
            const f2 fac = make_float2(__shfl_sync(kFull, lut_upd, code[2 * h] | (uint32_t)(r << LV)),
                                       __shfl_sync(kFull, lut_upd, code[2 * h + 1] | (uint32_t)(r << LV)));
            out[h] = fma2(nq[h], fac, base_t);
          }
        } else {
          const float srt = __fmul_rn(sqrt_fast(vzero ? 0.f : sv_raw), sc.rsqrt_bc2);
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const f2 sq = make_float2(sqrt_fast(__uint_as_float(Sr<BV>::floor_bits + (code[2 * h] << Sr<BV>::sh))),
                                      sqrt_fast(__uint_as_float(Sr<BV>::floor_bits + (code[2 * h + 1] << Sr<BV>::sh))));
            const f2 den = fma2(sq, splat(srt), splat(sc.eps));
            const f2 base_t = fma2(th[r][h], splat(nlrwd), th[r][h]);
            out[h] = fma2(mul2(nq[h], splat(unit)), make_float2(rcp_fast(den.x), rcp_fast(den.y)), base_t);
          }
        }
      } else {
        // d(x) = split logarithm of x / hi, clamped to [-W, 0]; code - K = round-half-even(d * K / W)
        const uint32_t ebase = kMagicBits - (vzero ? (uint32_t)kZeroBlockExp : (mxv[r] >> 23));
        [[maybe_unused]] const float half_step = tsHalf[r];
        [[maybe_unused]] const float srt_hi = __fmul_rn(sqrt_fast(vzero ? 0.f : sv_raw), sc.rsqrt_bc2);
        [[maybe_unused]] const float den_lo = __fmaf_rn(sqrt_fast(tsLo[r]), sc.rsqrt_bc2, sc.eps);
        uint32_t x[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint32_t b0 = __float_as_uint(vt[r][h].x), b1 = __float_as_uint(vt[r][h].y);
          const f2 de = add2(bits2(ebase + (b0 >> 23), ebase + (b1 >> 23)), splat(-kMagic));
          const f2 dp = fma2(lg_poly_pair(b0, b1), one2, splat(-tsPhi[r]));
          f2 d = add2(de, dp);
          d = make_float2(fminf(fmaxf(d.x, -tsW[r]), 0.0f), fminf(fmaxf(d.y, -tsW[r]), 0.0f));
          const f2 t = fma2(d, splat(tsInv[r]), splat(kMagic));
          x[2 * h] = __float_as_uint(t.x);
          x[2 * h + 1] = __float_as_uint(t.y);
          if constexpr (BV <= 4) {
            // the new code picks its level's factor from the lane table
            constexpr uint32_t bias = kMagicBits - (uint32_t)K;
            const f2 fac = make_float2(__shfl_sync(kFull, lut_upd, (int)((x[2 * h] - bias) | (uint32_t)(r << LV))),
                                       __shfl_sync(kFull, lut_upd, (int)((x[2 * h + 1] - bias) | (uint32_t)(r << LV))));
            out[h] = fma2(nq[h], fac, fma2(th[r][h], splat(nlrwd), th[r][h]));
            continue;
          }
          // sqrt of the decoded level: sqrt(hi) * 2^((code-K) * W/K / 2), or sqrt(lo) for code 0
          const f2 rr = add2(t, splat(-kMagic));
          const f2 arg = mul2(rr, splat(half_step));
          f2 den = fma2(make_float2(ex2_fast(arg.x), ex2_fast(arg.y)), splat(srt_hi), splat(sc.eps));
          den = make_float2(rr.x == -(float)K ? den_lo : den.x, rr.y == -(float)K ? den_lo : den.y);
          const f2 base_t = fma2(th[r][h], splat(nlrwd), th[r][h]);
          out[h] = fma2(mul2(nq[h], splat(unit)), make_float2(rcp_fast(den.x), rcp_fast(den.y)), base_t);
        }
        pack_store_row<BV>(vrow, lane, x, kMagicBits - (uint32_t)K);
      }
      *reinterpret_cast<float4*>(param + r * kRowElems) = make_float4(out[0].x, out[0].y, out[1].x, out[1].y);
      if constexpr (AMP) {
        if (ti.lp != nullptr) {
          const float o4[4] = {out[0].x, out[0].y, out[1].x, out[1].y};
          *reinterpret_cast<uint2*>(ti.lp + (row0 + r) * kRowElems + 4 * lane) = pack_lp(o4, lp_dtype);
        }
      }
    }
  }

  if (part != nullptr) {
    const float s0 = a0.x + a0.y, s1 = a1.x + a1.y, s2 = a2.x + a2.y;
    const bool hi = lane & 16;
    float x = (hi ? s2 : s0) + __shfl_xor_sync(kFull, hi ? s0 : s2, 16);
    float y = (hi ? 0.f : s1) + __shfl_xor_sync(kFull, hi ? s1 : 0.f, 16);
    const bool q = lane & 8;
    float z = (q ? y : x) + __shfl_xor_sync(kFull, q ? x : y, 8);
    z += __shfl_xor_sync(kFull, z, 4);
    z += __shfl_xor_sync(kFull, z, 2);
    z += __shfl_xor_sync(kFull, z, 1);
    if ((lane & 7) == 0 && lane < 24) part[lane >> 3] = (double)z;
  }
}

template <int GDT, bool AMP>
__device__ __forceinline__ void dispatch_variant(const uint8_t* __restrict__ stage, const TileInfo& ti, const StepConsts& sc,
                                                 int lane, int warp, uint32_t ebar, double* __restrict__ part, float grad_mul) {
#define STQ_VCASE(IM, IV, BM, BV, VM) \
  case IM * 10 + IV: tile_body_var<BM, BV, VM, GDT, AMP>(stage, ti, sc, lane, warp, ebar, part, grad_mul); break;
#define STQ_VCASES_M(IM, BM)                                                                              \
  STQ_VCASE(IM, 0, BM, 2, 2) STQ_VCASE(IM, 1, BM, 3, 2) STQ_VCASE(IM, 2, BM, 4, 2) STQ_VCASE(IM, 3, BM, 8, 2) \
  STQ_VCASE(IM, 4, BM, 16, 2) STQ_VCASE(IM, 5, BM, 2, 3) STQ_VCASE(IM, 6, BM, 3, 3) STQ_VCASE(IM, 7, BM, 4, 3) \
  STQ_VCASE(IM, 8, BM, 8, 3) STQ_VCASE(IM, 9, BM, 16, 3)
  switch ((ti.packed & 0xFFu) * 10 + (((ti.packed >> 8) & 0xFFu) - 7u)) {
    STQ_VCASES_M(0, 2)
    STQ_VCASES_M(1, 3)
    STQ_VCASES_M(2, 4)
    STQ_VCASES_M(3, 8)
    STQ_VCASES_M(4, 16)
    default: break;
  }
#undef STQ_VCASES_M
#undef STQ_VCASE
}

// Calls f with the width behind a width index as a compile-time constant (warp-uniform switch).
template <class F>
__device__ __forceinline__ void with_m_width(uint32_t idx, F&& f) {
  switch (idx) {
    case 0: f(std::integral_constant<int, 2>{}); break;
    case 1: f(std::integral_constant<int, 3>{}); break;
    case 2: f(std::integral_constant<int, 4>{}); break;
    case 3: f(std::integral_constant<int, 8>{}); break;
    default: f(std::integral_constant<int, 16>{}); break;
  }
}
template <class F>
__device__ __forceinline__ void with_v_width(uint32_t idx, F&& f) {   // f(width, piecewise-linear variant?)
  switch (idx) {
    case 0: f(std::integral_constant<int, 2>{}, std::false_type{}); break;
    case 1: f(std::integral_constant<int, 3>{}, std::false_type{}); break;
    case 2: f(std::integral_constant<int, 4>{}, std::false_type{}); break;
    case 3: f(std::integral_constant<int, 8>{}, std::false_type{}); break;
    case 4: f(std::integral_constant<int, 16>{}, std::false_type{}); break;
    case 5: f(std::integral_constant<int, 8>{}, std::true_type{}); break;
    default: f(std::integral_constant<int, 16>{}, std::true_type{}); break;
  }
}

// A tile whose tensor changes width inside the step (Algorithm 1 writes the states of a decision step
// at the new widths): the stored widths and the widths to write are runtime values here, so every
// row decode and encode goes through a warp-uniform switch into the same specialised row functions
// the fused bodies use.  One body serves all combinations; it is slower than a fused body and far
// faster than leaving these tiles to the generic kernel.
template <int GDT, bool AMP>
__device__ __forceinline__ void tile_body_split(const uint8_t* __restrict__ stage, const TileInfo& ti, const StepConsts& sc,
                                             const float* __restrict__ lut8, int lane, int warp, uint32_t empty_bar,
                                             double* __restrict__ part, float grad_mul) {
  const uint32_t* lutn = reinterpret_cast<const uint32_t*>(lut8 + 256);
  const int lgB = (int)((ti.packed >> 16) & 0xFFu);
  [[maybe_unused]] const uint32_t lp_dtype = ti.packed >> 24;
  const uint32_t im = ti.packed & 0xFFu, iv = (ti.packed >> 8) & 0xFFu;
  const uint32_t om = ti.out & 0xFFu, ov = (ti.out >> 8) & 0xFFu;
  const uint32_t bm_out = om == 0 ? 2u : om == 1 ? 3u : om == 2 ? 4u : om == 3 ? 8u : 16u;
  const float qmax_out = (float)((1u << (bm_out - 1u)) - 1u);
  const float lrwd = sc.l2_mode ? 0.0f : ti.wdx;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f;

#pragma unroll 1
  for (int pass = 0; pass < R / RP; ++pass) {
    const int row0 = warp * R + pass * RP;
    float th[RP][4], g[RP][4], mt[RP][4], vt[RP][4];
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      const int row = row0 + r;
      const int elem = row * kRowElems + 4 * lane;
      const float4 t4 = *reinterpret_cast<const float4*>(stage + kOffTheta + 4 * elem);
      th[r][0] = t4.x; th[r][1] = t4.y; th[r][2] = t4.z; th[r][3] = t4.w;
      lds_grad<GDT>(stage, elem, g[r]);
      const int blk = (row * kRowElems) >> lgB;
      const float sm = *reinterpret_cast<const float*>(stage + kOffMs + 4 * blk);
      const float sv = *reinterpret_cast<const float*>(stage + kOffVs + 4 * blk);
      with_m_width(im, [&](auto B) {
        uint32_t w[2];
        lds_codes<decltype(B)::value>(stage + kOffMc + row * (16 * decltype(B)::value), lane, w);
        decode_lin_row<decltype(B)::value>(w, sm, mt[r]);
      });
      with_v_width(iv, [&](auto B, auto pl) {
        uint32_t w[2];
        lds_codes<decltype(B)::value>(stage + kOffVc + row * (16 * decltype(B)::value), lane, w);
        if constexpr (decltype(pl)::value) decode_pl_row<decltype(B)::value>(w, __float_as_uint(sv), lutn, vt[r]);
        else decode_log_row<decltype(B)::value>(w, sv, lut8, vt[r]);
      });
    }
    if (pass == R / RP - 1) {
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar);
    }
    if constexpr (AMP) {
#pragma unroll
      for (int r = 0; r < RP; ++r)
#pragma unroll
        for (int k = 0; k < 4; ++k) g[r][k] = __fmul_rn(g[r][k], grad_mul);
    }
    if (part != nullptr) {
#pragma unroll
      for (int r = 0; r < RP; ++r)
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          a0 += g[r][k];
          a1 += fabsf(g[r][k]);
          a2 = __fmaf_rn(g[r][k], g[r][k], a2);
        }
    }
    if (sc.l2_mode) {
#pragma unroll
      for (int r = 0; r < RP; ++r)
#pragma unroll
        for (int k = 0; k < 4; ++k) g[r][k] = __fadd_rn(g[r][k], __fmul_rn(ti.wdx, th[r][k]));
    }
#pragma unroll
    for (int r = 0; r < RP; ++r)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float gk = g[r][k];
        mt[r][k] = __fmaf_rn(sc.b1, mt[r][k], __fmul_rn(sc.c1, gk));
        vt[r][k] = __fmaf_rn(sc.b2, vt[r][k], __fmul_rn(__fmul_rn(sc.c2, gk), gk));
      }
    uint32_t mxm[RP], mxv[RP];
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      const float am = fmaxf(fmaxf(fabsf(mt[r][0]), fabsf(mt[r][1])), fmaxf(fabsf(mt[r][2]), fabsf(mt[r][3])));
      const float av = fmaxf(fmaxf(vt[r][0], vt[r][1]), fmaxf(vt[r][2], vt[r][3]));
      mxm[r] = __reduce_max_sync(kFull, __float_as_uint(am));
      mxv[r] = __reduce_max_sync(kFull, __float_as_uint(av));
    }
    if (RP >= 2 && lgB >= 8) {
#pragma unroll
      for (int r = 0; r + 1 < RP; r += 2) {
        mxm[r] = mxm[r + 1] = max(mxm[r], mxm[r + 1]);
        mxv[r] = mxv[r + 1] = max(mxv[r], mxv[r + 1]);
      }
    }
    float* param = ti.param + row0 * kRowElems + 4 * lane;
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      const int row = row0 + r;
      const float sm_raw = __uint_as_float(mxm[r]);
      const bool mzero = sm_raw < kTiny;
      const float sv_raw = __uint_as_float(mxv[r]);
      const bool vzero = sv_raw < kTiny;
      const float s_v = vzero ? 0.f : sv_raw;
      // (this body computes the block constants in every lane: it runs on decision steps only)
      const float inv_m = mzero ? 0.f : __fmul_rn(qmax_out, __frcp_rn(sm_raw));
      float mq[4], vq[4];
      with_m_width(om, [&](auto B) {
        encode_lin_row<decltype(B)::value>(ti.mco + row * (16 * decltype(B)::value), lane, mt[r], __fmul_rn(sm_raw, sc.step_size), inv_m, mq);
      });
      with_v_width(ov, [&](auto B, auto pl) {
        uint8_t* dst = ti.vco + row * (16 * decltype(B)::value);
        if constexpr (decltype(pl)::value) {
          encode_pl_row<decltype(B)::value>(dst, lane, vt[r], vzero ? 0x7F800000u : mxv[r], vzero ? 0u : mxv[r], lutn, vq);
        } else if constexpr (decltype(B)::value <= 4) {
          const float c = vzero ? 0.f : __fmul_rn(kSqrt2, __frcp_rn(sv_raw));
          encode_log_row<decltype(B)::value>(dst, lane, vt[r], s_v, c, 0u, lut8, vq);
        } else {
          const uint32_t ebase = kMagicBits - (vzero ? (uint32_t)kZeroBlockExp : (mxv[r] >> 23));
          encode_log_row<decltype(B)::value>(dst, lane, vt[r], s_v, lg_poly(mxv[r]), ebase, lut8, vq);
        }
      });
      const int e_row = row * kRowElems;
      if (lane == 0 && (e_row & ((1 << lgB) - 1)) == 0) {
        ti.mso[e_row >> lgB] = mzero ? 0.f : sm_raw;
        ti.vso[e_row >> lgB] = s_v;
      }
      float out[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float den = __fmaf_rn(sqrt_fast(vq[k]), sc.rsqrt_bc2, sc.eps);
        const float upd = __fmul_rn(mq[k], rcp_fast(den));
        out[k] = __fadd_rn(th[r][k], -__fmaf_rn(th[r][k], lrwd, upd));
      }
      *reinterpret_cast<float4*>(param + r * kRowElems) = make_float4(out[0], out[1], out[2], out[3]);
      if constexpr (AMP) {
        if (ti.lp != nullptr)
          *reinterpret_cast<uint2*>(ti.lp + row * kRowElems + 4 * lane) = pack_lp(out, lp_dtype);
      }
    }
  }
  if (part != nullptr) {
    const bool hi = lane & 16;
    float x = (hi ? a2 : a0) + __shfl_xor_sync(kFull, hi ? a0 : a2, 16);
    float y = (hi ? 0.f : a1) + __shfl_xor_sync(kFull, hi ? a1 : 0.f, 16);
    const bool q = lane & 8;
    float z = (q ? y : x) + __shfl_xor_sync(kFull, q ? x : y, 8);
    z += __shfl_xor_sync(kFull, z, 4);
    z += __shfl_xor_sync(kFull, z, 2);
    z += __shfl_xor_sync(kFull, z, 1);
    if ((lane & 7) == 0 && lane < 24) part[lane >> 3] = (double)z;
  }
}

// Scheduling: the fast tiles are grouped by body (width pair and variant of the v code).  A CTA starts in the group
// the host assigned to it and takes chunks of consecutive tiles (kFastChunk of them, single tiles when the
// launch is small) from that group's
// counter; when its group runs dry it moves on to the one with the most tiles left.  So a CTA runs
// few different bodies (a change of body is an instruction-cache refill), the tiles of a group are
// streamed together, and the balance is dynamic.
__device__ __forceinline__ uint32_t width_index(uint32_t b) { return b == 2 ? 0u : b == 3 ? 1u : b == 4 ? 2u : b == 8 ? 3u : 4u; }

// AMP: the mixed-precision extras (gradient unscaling, low-precision parameter copy) are compiled
// in only for launches that use them, so the plain step pays nothing for them.
// LIST: which work list the launch serves, each compiled apart so that none disturbs the register allocation
// of another: 0 the fused bodies of the default and "pl" codes, 1 the fused bodies of the "sr" and "ts" codes
// of the second moment, 2 the tiles of tensors that change width inside the step (one runtime-width body).
template <int GDT, bool AMP, int LIST>
__global__ void __launch_bounds__(kFastThreads, kFastCtasPerSm)
stq_step_fast_kernel(const TensorDesc* __restrict__ table, const uint32_t* __restrict__ tile_map,
                     FastSched* __restrict__ sched, const StepConsts sc_in, double* __restrict__ partials,
                     int* __restrict__ err_flag) {
  // The launches with the mixed-precision extras also accept the step's scalars from device memory
  // (a step count and learning rate that advance between replays of a captured graph).
  StepConsts sc_dev;
  const StepConsts* scp = &sc_in;
  if constexpr (AMP) {
    if (sc_in.dev_scalars != nullptr) {
      sc_dev = sc_in;
      sc_dev.step_size = __ldg(sc_in.dev_scalars + 0);
      sc_dev.rsqrt_bc2 = __ldg(sc_in.dev_scalars + 1);
      sc_dev.lr = (double)__ldg(sc_in.dev_scalars + 2);
      scp = &sc_dev;
    }
  }
  const StepConsts& sc = *scp;
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t full0 = smem_u32(smem + kOffBars);
  const uint32_t empty0 = full0 + 8 * kStages;
  float* lut8 = reinterpret_cast<float*>(smem + kOffLut);
  constexpr uint32_t kEnd = 0xFFFFFFFFu;   // TileInfo.tile of the closing stage
  constexpr uint32_t gsz = GDT == 0 ? 4u : 2u;
  // a non-finite gradient somewhere in the model: the whole step is skipped (every thread sees the same value)
  if (sc.found_inf != nullptr && __ldg(sc.found_inf) != 0.0f) return;
  const float grad_mul = sc.inv_scale != nullptr ? __ldg(sc.inv_scale) : 1.0f;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, kConsumerWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (tid < 256) {   // decode table of the 8-bit log code: ex((q - 255) * fl(30/255))
    constexpr float cb = (float)Wd<8>::Roct / (float)Wd<8>::K;
    lut8[tid] = ex2_poly(__fmul_rn((float)(tid - 255), cb));
    reinterpret_cast<uint32_t*>(lut8 + 256)[tid] = pl_below<8>((uint32_t)tid);
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ================================ producer ========================================================
    if (lane != 0) return;
    const uint32_t ng = sched->ng, chunk = sched->chunk;
    uint32_t grp = sched->cta_group[blockIdx.x];
    uint32_t issued = 0;
    int s = 0;
    uint32_t phase = 0;        // parity of the use of stage s that is being filled
    uint32_t last_use[kStages];   // parity of the latest fill of each stage (2: never filled)
#pragma unroll
    for (int k = 0; k < kStages; ++k) last_use[k] = 2u;
    bool ok = true;
    while (ok) {
      const uint32_t gbeg = sched->grp_begin[grp], gend = sched->grp_begin[grp + 1];
      const uint32_t c = atomicAdd(&sched->ctr[grp], 1u);
      const unsigned long long t0 = (unsigned long long)gbeg + (unsigned long long)c * chunk;
      if (t0 >= gend) {
        // This group has been handed out completely.  Move to the group with the most tiles left (a change
        // of body is an instruction-cache refill: better paid once, for a long stay); none left: done.
        // The counters only grow, so a group seen empty stays empty and no tile is missed.
        uint32_t best = 0u, best_left = 0u;
        for (uint32_t k = 0; k < ng; ++k) {
          const unsigned long long size = sched->grp_begin[k + 1] - sched->grp_begin[k];
          const unsigned long long taken = (unsigned long long)*reinterpret_cast<volatile uint32_t*>(&sched->ctr[k]) * chunk;
          const uint32_t left = taken < size ? (uint32_t)(size - taken) : 0u;
          if (left > best_left) { best_left = left; best = k; }
        }
        if (best_left == 0u) break;
        grp = best;
        continue;
      }
      const uint32_t t1 = (uint32_t)(t0 + chunk < gend ? t0 + chunk : gend);
      for (uint32_t tile = (uint32_t)t0; tile < t1; ++tile) {
        // Everything that can be prepared without the stage (table look-ups, addresses) comes before the
        // wait for it, so that the copies leave the moment the consumers release the stage: in the
        // memory-bound bodies the time from release to issue adds to every tile's turnaround.
        const TensorDesc* T = table + __ldg(tile_map + tile);
        const unsigned long long e0 = (unsigned long long)(tile - T->tile0) * kTile;
        const uint32_t bm = T->bm_in, bv = T->bv_in, bmo = T->bm_out, bvo = T->bv_out;
        const uint32_t lgB = T->block == 128 ? 7u : T->block == 256 ? 8u : 9u;
        const uint32_t nb_m = (kTile / 8) * bm, nb_v = (kTile / 8) * bv, nb_s = (uint32_t)(kTile * 4) >> lgB;
        const uint32_t vmode = LIST == 1 ? T->v_mode : (T->v_mode & 1u);
        const uint32_t spb = vmode == 3u ? 2u : 1u;          // scales per block of v: two in the two-scale code
        TileInfo ti;
        ti.param = T->param + e0;
        ti.mco = T->mc_out + (e0 >> 3) * bmo;
        ti.vco = T->vc_out + (e0 >> 3) * bvo;
        ti.mso = T->ms_out + (e0 >> lgB);
        ti.vso = T->vs_out + spb * (e0 >> lgB);
        ti.lp = T->param_lp ? reinterpret_cast<uint16_t*>(T->param_lp) + e0 : nullptr;
        // v index: 0..4 the widths in the default code, 5, 6: 8 and 16 bits in the "pl" code, 7..11 the widths in the
        // "sr" code, 12..16 in the "ts" code
        const uint32_t iv = vmode >= 2u ? width_index(bv) + (vmode == 2u ? 7u : 12u)
                                        : width_index(bv) + (vmode == 1u && bv >= 8u ? 2u : 0u);
        ti.packed = width_index(bm) | (iv << 8) | (lgB << 16) | (T->lp_dtype << 24);
        ti.wdx = sc.l2_mode ? T->wd : (float)(sc.lr * (double)T->wd);
        ti.tile = tile;
        ti.out = width_index(bmo) | ((width_index(bvo) + (vmode == 1u && bvo >= 8u ? 2u : 0u)) << 8);
        ti.sr_key = LIST == 1 ? mix32(mix32(T->sr_id ^ sc.sr_h) + (uint32_t)(e0 >> 32)) : 0u;
        ti.e0 = (uint32_t)e0;
        ti.pad[0] = ti.pad[1] = 0u;
        const uint8_t* src_g = reinterpret_cast<const uint8_t*>(T->grad) + e0 * gsz;
        const uint8_t* src_mc = T->mc_in + (e0 >> 3) * bm;
        const uint8_t* src_vc = T->vc_in + (e0 >> 3) * bv;
        const float* src_ms = T->ms_in + (e0 >> lgB);
        const float* src_vs = T->vs_in + spb * (e0 >> lgB);
        if (issued >= (uint32_t)kStages && !mbar_wait(empty0 + 8 * s, phase ^ 1u)) { ok = false; break; }
        *reinterpret_cast<TileInfo*>(smem + kOffInfo + kInfoBytes * s) = ti;
        const uint32_t bar = full0 + 8 * s;
        const uint32_t dst = smem_u32(smem + s * kStageBytes);
        mbar_expect_tx(bar, kTile * 4 + kTile * gsz + nb_m + nb_v + (1u + spb) * nb_s);
        bulk_g2s(dst + kOffTheta, ti.param, kTile * 4, bar);
        bulk_g2s(dst + kOffGrad, src_g, kTile * gsz, bar);
        bulk_g2s(dst + kOffMc, src_mc, nb_m, bar);
        bulk_g2s(dst + kOffVc, src_vc, nb_v, bar);
        bulk_g2s(dst + kOffMs, src_ms, nb_s, bar);
        bulk_g2s(dst + kOffVs, src_vs, spb * nb_s, bar);
        ++issued;
#pragma unroll
        for (int k = 0; k < kStages; ++k)
          if (k == s) last_use[k] = phase;
        if (++s == kStages) { s = 0; phase ^= 1u; }
      }
    }
    // Closing stage: tells the consumers that no tile follows.  Its turn comes only after the
    // consumers have released the stage, i.e. after every copy issued into it has landed and been
    // read.  After a time-out the copies still in flight get one more bounded wait instead, so that
    // none lands in shared memory that no longer belongs to this CTA.
    if (ok && issued >= (uint32_t)kStages) ok = mbar_wait(empty0 + 8 * s, phase ^ 1u);
    // The last producer to get here leaves the work list as the next launch wants to find it.
    __threadfence();
    if (atomicAdd(&sched->done, 1u) == gridDim.x - 1u) {
      for (uint32_t k = 0; k < ng; ++k) sched->ctr[k] = 0u;
      sched->done = 0u;
    }
    if (ok) {
      reinterpret_cast<TileInfo*>(smem + kOffInfo + kInfoBytes * s)->tile = kEnd;
      mbar_arrive(full0 + 8 * s);
    } else {
      atomicExch(err_flag, 1);
#pragma unroll
      for (int k = 0; k < kStages; ++k)
        if (last_use[k] != 2u) mbar_wait(full0 + 8 * k, last_use[k]);
    }
    return;
  }

  // ================================== consumers =========================================================
  int s = 0;
  uint32_t phase = 0;
  while (true) {
    if (!mbar_wait(full0 + 8 * s, phase)) {
      if (lane == 0) atomicExch(err_flag, 1);
      break;
    }
    const uint8_t* stage = smem + s * kStageBytes;
    const TileInfo ti = *reinterpret_cast<const TileInfo*>(smem + kOffInfo + kInfoBytes * s);
    if (ti.tile == kEnd) break;
    const uint32_t ebar = empty0 + 8 * s;
    double* part = partials ? partials + ((size_t)ti.tile * kConsumerWarps + warp) * 3 : nullptr;

#define STQ_CASE(IM, IV, BM, BV, VPL) \
  case IM * 7 + IV: tile_body<BM, BV, VPL, GDT, AMP>(stage, ti, sc, lut8, lane, warp, ebar, part, grad_mul); break;
#define STQ_CASES_M(IM, BM)                                                                                   \
  STQ_CASE(IM, 0, BM, 2, false) STQ_CASE(IM, 1, BM, 3, false) STQ_CASE(IM, 2, BM, 4, false) STQ_CASE(IM, 3, BM, 8, false) \
  STQ_CASE(IM, 4, BM, 16, false) STQ_CASE(IM, 5, BM, 8, true) STQ_CASE(IM, 6, BM, 16, true)
    if constexpr (LIST == 2) {
      tile_body_split<GDT, AMP>(stage, ti, sc, lut8, lane, warp, ebar, part, grad_mul);
    } else if constexpr (LIST == 1) {
      dispatch_variant<GDT, AMP>(stage, ti, sc, lane, warp, ebar, part, grad_mul);
    } else {
      switch ((ti.packed & 0xFFu) * 7 + ((ti.packed >> 8) & 0xFFu)) {
        STQ_CASES_M(0, 2)
        STQ_CASES_M(1, 3)
        STQ_CASES_M(2, 4)
        STQ_CASES_M(3, 8)
        STQ_CASES_M(4, 16)
        default: break;
      }
    }
    if (++s == kStages) { s = 0; phase ^= 1u; }
  }
}

template <int GDT, bool AMP, int LIST>
cudaError_t launch_fast_t(const TensorDesc* table, const uint32_t* tile_map, FastSched* sched, const StepConsts& sc,
                          double* partials, int* err_flag, int grid, cudaStream_t stream) {
  auto kern = stq_step_fast_kernel<GDT, AMP, LIST>;
  // per device and cheap, so simply repeated: the kernel needs more than the default 48 KB
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  // (the group counters are zero: uploaded so, and every launch resets them on its way out)
  kern<<<grid, kFastThreads, kSmemBytes, stream>>>(table, tile_map, sched, sc, partials, err_flag);
  return cudaGetLastError();
}


}  // namespace
}  // namespace stq

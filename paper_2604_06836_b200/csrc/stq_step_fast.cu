// The main kernel of the quantized AdamW step: full tiles of tensors whose widths stay the same
// this step (2..16 bits).  Everything else (ragged last tiles, 32-bit states, width changes inside
// the step, init, repack) goes through the generic kernel in stq_kernels.cu.
//
// Data movement: a persistent CTA walks its tiles through a two-stage shared-memory ring.  One
// elected thread issues, per tile, four bulk asynchronous copies (parameters, gradients, m codes,
// v codes: each a contiguous, 16-byte aligned range because a tile starts at a multiple of 1024
// elements) that complete on an mbarrier; the eight warps wait on the barrier, pull their rows into
// registers with conflict-free 128/64/32-bit shared loads, and release the stage right away, so the
// copies of the tile after next are in flight while this tile is computed.  Results go straight
// from registers to global memory with 128-bit (parameters) and 8..64-bit (codes) stores.  Every
// wait on a barrier is bounded; on expiry the kernel raises an error flag and returns.
//
// Arithmetic: identical to the generic kernel (same roundings, see there), specialised per width
// so that shifts and masks are immediates, with the per-block constants (one division, one
// reciprocal or logarithm of the block maximum) computed by one lane per row and broadcast.
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
constexpr int kStages = 2;
constexpr int kOffTheta = 0;
constexpr int kOffGrad = 4 * kTile;
constexpr int kOffMc = 8 * kTile;
constexpr int kOffVc = 10 * kTile;
constexpr int kStageBytes = 12 * kTile;
constexpr int kSmemBytes = kStages * kStageBytes + 64;
constexpr long long kWaitCycles = 4000000000ll;   // ~2 s: far beyond any copy; then give up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// Bounded wait: returns false if the phase did not complete within kWaitCycles.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kWaitCycles) return false;
  }
  return true;
}
// 1-D bulk copy global -> shared of this CTA, completion counted in bytes on `bar`.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
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
__device__ __forceinline__ void decode_log_row(const uint32_t (&w)[2], float s, float (&out)[4]) {
  if constexpr (B <= 4) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t c = (w[0] >> (B * k)) & Wd<B>::mask;
      out[k] = __fmul_rn(s, __uint_as_float((c + (uint32_t)(127 - Wd<B>::K)) << 23));
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

// Packs x_k = base + u_k into the lane's field(s) and stores them.  row_ptr: the row's codes in
// global memory.
template <int B>
__device__ __forceinline__ void pack_store_row(uint8_t* row_ptr, int lane, const uint32_t (&x)[4], uint32_t base) {
  if constexpr (B == 2) {
    const uint32_t w = x[0] + (x[1] << 2) + (x[2] << 4) + (x[3] << 6) - base * Wd<2>::fieldsum;
    *(row_ptr + lane) = (uint8_t)w;
  } else if constexpr (B == 3) {
    const uint32_t p = (x[0] + (x[1] << 3) + (x[2] << 6) + (x[3] << 9) - base * Wd<3>::fieldsum) & 0xFFFu;
    const int first = (8 * lane) / 3;
    uint32_t w = 0u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int src = first + i;
      uint32_t v = __shfl_sync(kFull, p, src & 31);
      const int sh = 12 * src - 32 * lane;
      if (sh >= 32) v = 0u;
      else if (sh >= 0) v <<= sh;
      else v >>= -sh;
      w |= v;
    }
    if (lane < 12) *reinterpret_cast<uint32_t*>(row_ptr + 4 * lane) = w;
  } else if constexpr (B == 4) {
    const uint32_t w = x[0] + (x[1] << 4) + (x[2] << 8) + (x[3] << 12) - base * Wd<4>::fieldsum;
    *reinterpret_cast<uint16_t*>(row_ptr + 2 * lane) = (uint16_t)w;
  } else if constexpr (B == 8) {
    const uint32_t w = x[0] + (x[1] << 8) + (x[2] << 16) + (x[3] << 24) - base * Wd<8>::fieldsum;
    *reinterpret_cast<uint32_t*>(row_ptr + 4 * lane) = w;
  } else {
    const uint32_t w0 = x[0] + (x[1] << 16) - base * Wd<16>::fieldsum;
    const uint32_t w1 = x[2] + (x[3] << 16) - base * Wd<16>::fieldsum;
    *reinterpret_cast<uint2*>(row_ptr + 8 * lane) = make_uint2(w0, w1);
  }
}

// Quantize one row of new first moments, store the codes, return the decoded values.
template <int B>
__device__ __forceinline__ void encode_lin_row(uint8_t* row_ptr, int lane, const float (&m)[4], float s, float inv,
                                               float (&mq)[4]) {
  constexpr float invq = 1.0f / (float)Wd<B>::qmax;
  constexpr float mg = kMagic + (float)Wd<B>::half;
  uint32_t x[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float t = __fmaf_rn(m[k], inv, mg);
    x[k] = __float_as_uint(t);
    mq[k] = __fmul_rn(s, __fmul_rn(__fadd_rn(t, -mg), invq));
  }
  pack_store_row<B>(row_ptr, lane, x, kMagicBits);
}

// Per-block constants of the log quantizer: octave widths need c = sqrt2/s, the others E_s and P(s).
struct LogBlock {
  float s;      // stored scale (0 for a zero block)
  float c;      // octave widths: fl(fl(1/s)*sqrt2), 0 for a zero block
  float Ps;     // 8/16 bit: P(s)
  uint32_t ebase;   // 8/16 bit: kMagicBits - E_s
};

template <int B>
__device__ __forceinline__ void encode_log_row(uint8_t* row_ptr, int lane, const float (&v)[4], const LogBlock& lb,
                                               float (&vq)[4]) {
  uint32_t x[4];
  if constexpr (B <= 4) {
    constexpr uint32_t emin = (uint32_t)(127 - Wd<B>::K);
    const float ymin = __uint_as_float(emin << 23);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t yb = __float_as_uint(fmaxf(__fmul_rn(v[k], lb.c), ymin));
      x[k] = yb >> 23;
      vq[k] = __fmul_rn(lb.s, __uint_as_float(yb & 0x7F800000u));
    }
    pack_store_row<B>(row_ptr, lane, x, emin);
  } else {
    constexpr float a = (float)Wd<B>::K / (float)Wd<B>::Roct;
    constexpr float cb = (float)Wd<B>::Roct / (float)Wd<B>::K;
    constexpr float negR = -(float)Wd<B>::Roct;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t xb = __float_as_uint(v[k]);
      const float de = __fadd_rn(__uint_as_float(lb.ebase + (xb >> 23)), -kMagic);
      const float dp = __fadd_rn(lg_poly(xb), -lb.Ps);
      const float d = fmaxf(__fadd_rn(de, dp), negR);
      const float t = __fmaf_rn(d, a, kMagic);
      x[k] = __float_as_uint(t);
      vq[k] = __fmul_rn(lb.s, ex2_poly(__fmul_rn(__fadd_rn(t, -kMagic), cb)));
    }
    pack_store_row<B>(row_ptr, lane, x, kMagicBits - (uint32_t)Wd<B>::K);
  }
}

template <int GDT>
__device__ __forceinline__ void lds_grad(const uint8_t* stage, int elem, float (&g)[4]) {
  if constexpr (GDT == 0) {
    const float4 v = *reinterpret_cast<const float4*>(stage + kOffGrad + 4 * elem);
    g[0] = v.x; g[1] = v.y; g[2] = v.z; g[3] = v.w;
  } else {
    const uint2 v = *reinterpret_cast<const uint2*>(stage + kOffGrad + 2 * elem);
    g[0] = __uint_as_float(v.x << 16);
    g[1] = __uint_as_float(v.x & 0xFFFF0000u);
    g[2] = __uint_as_float(v.y << 16);
    g[3] = __uint_as_float(v.y & 0xFFFF0000u);
  }
}

#define STQ_WIDTH_SWITCH(bits, CALL)           \
  switch (bits) {                              \
    case 2: { CALL(2); } break;                \
    case 3: { CALL(3); } break;                \
    case 4: { CALL(4); } break;                \
    case 8: { CALL(8); } break;                \
    default: { CALL(16); } break;              \
  }

template <int GDT, bool STATS>
__global__ void __launch_bounds__(kThreads, kFastCtasPerSm)
stq_step_fast_kernel(const TensorDesc* __restrict__ table, const uint32_t* __restrict__ tile_map, uint32_t n_fast,
                     const StepConsts sc, double* __restrict__ partials, int* __restrict__ err_flag) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ double s_part[kThreads / 32][3];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t bar0 = smem_u32(smem + kStages * kStageBytes);
  const uint32_t first = blockIdx.x, stride = gridDim.x;
  if (first >= n_fast) return;
  const uint32_t n_my = (n_fast - first + stride - 1) / stride;
  constexpr uint32_t gsz = GDT == 0 ? 4u : 2u;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  // thread 0: start the copies of one tile into stage s
  auto issue = [&](uint32_t it, int s) {
    const uint32_t tile = first + it * stride;
    const TensorDesc* T = table + __ldg(tile_map + tile);
    const unsigned long long e0 = (unsigned long long)(tile - T->tile0) * kTile;
    const uint32_t bm = T->bm_in, bv = T->bv_in;
    const uint32_t nb_m = (kTile / 8) * bm, nb_v = (kTile / 8) * bv;
    const uint32_t bar = bar0 + 8 * s;
    const uint32_t dst = smem_u32(smem + s * kStageBytes);
    mbar_expect_tx(bar, kTile * 4 + kTile * gsz + nb_m + nb_v);
    bulk_g2s(dst + kOffTheta, T->param + e0, kTile * 4, bar);
    bulk_g2s(dst + kOffGrad, reinterpret_cast<const uint8_t*>(T->grad) + e0 * gsz, kTile * gsz, bar);
    bulk_g2s(dst + kOffMc, T->mc_in + (e0 >> 3) * bm, nb_m, bar);
    bulk_g2s(dst + kOffVc, T->vc_in + (e0 >> 3) * bv, nb_v, bar);
  };
  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s)
      if ((uint32_t)s < n_my) issue(s, s);
  }

  uint32_t failed_at = 0xFFFFFFFFu;
  for (uint32_t it = 0; it < n_my; ++it) {
    const int s = it % kStages;
    const uint32_t parity = (it / kStages) & 1u;
    const uint32_t tile = first + it * stride;
    const TensorDesc* __restrict__ T = table + __ldg(tile_map + tile);
    const uint32_t e_warp = (tile - T->tile0) * (uint32_t)kTile + (uint32_t)warp * (R * kRowElems);   // fits: checked on the host
    const int bm = T->bm_in, bv = T->bv_in;
    const int lgB = 7 + (int)(T->block >> 8);
    const float* ms_in = T->ms_in;
    const float* vs_in = T->vs_in;
    float s_m_in[R], s_v_in[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const uint32_t blk = (e_warp + r * kRowElems) >> lgB;
      s_m_in[r] = __ldg(ms_in + blk);
      s_v_in[r] = __ldg(vs_in + blk);
    }

    // a thread whose wait ran out still reaches the barrier below, so the CTA gives up as one
    const bool landed = mbar_wait(bar0 + 8 * s, parity);

    // ---- staged tile -> registers ---------------------------------------------------------------------
    const uint8_t* stage = smem + s * kStageBytes;
    float th[R][4], g[R][4];
    uint32_t wm[R][2], wv[R][2];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int row = warp * R + r;
      const int elem = row * kRowElems + 4 * lane;
      const float4 t4 = *reinterpret_cast<const float4*>(stage + kOffTheta + 4 * elem);
      th[r][0] = t4.x; th[r][1] = t4.y; th[r][2] = t4.z; th[r][3] = t4.w;
      lds_grad<GDT>(stage, elem, g[r]);
    }
#define STQ_LDS_M(BW)                                                                   \
  _Pragma("unroll") for (int r = 0; r < R; ++r)                                         \
      lds_codes<BW>(stage + kOffMc + (warp * R + r) * (16 * BW), lane, wm[r]);
#define STQ_LDS_V(BW)                                                                   \
  _Pragma("unroll") for (int r = 0; r < R; ++r)                                         \
      lds_codes<BW>(stage + kOffVc + (warp * R + r) * (16 * BW), lane, wv[r]);
    STQ_WIDTH_SWITCH(bm, STQ_LDS_M)
    STQ_WIDTH_SWITCH(bv, STQ_LDS_V)

    // the stage is free again: everyone has its data in registers
    if (__syncthreads_or(!landed)) {
      failed_at = it;
      break;
    }
    if (tid == 0 && it + kStages < n_my) issue(it + kStages, s);

    // ---- decode, moments -------------------------------------------------------------------------------
    float mt[R][4], vt[R][4];
#define STQ_DEC_M(BW) \
  _Pragma("unroll") for (int r = 0; r < R; ++r) decode_lin_row<BW>(wm[r], s_m_in[r], mt[r]);
#define STQ_DEC_V(BW) \
  _Pragma("unroll") for (int r = 0; r < R; ++r) decode_log_row<BW>(wv[r], s_v_in[r], vt[r]);
    STQ_WIDTH_SWITCH(bm, STQ_DEC_M)
    STQ_WIDTH_SWITCH(bv, STQ_DEC_V)

    float st_g = 0.f, st_a = 0.f, st_q = 0.f;
    const float wd = T->wd;
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float gk = g[r][k];
        if constexpr (STATS) {
          st_g += gk;
          st_a += fabsf(gk);
          st_q = __fmaf_rn(gk, gk, st_q);
        }
        if (sc.l2_mode) gk = __fadd_rn(gk, __fmul_rn(wd, th[r][k]));
        mt[r][k] = __fadd_rn(__fmul_rn(sc.b1, mt[r][k]), __fmul_rn(sc.c1, gk));
        vt[r][k] = __fadd_rn(__fmul_rn(sc.b2, vt[r][k]), __fmul_rn(__fmul_rn(sc.c2, gk), gk));
      }
    }

    // ---- block maxima ----------------------------------------------------------------------------------
    uint32_t mxm[R], mxv[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const float am = fmaxf(fmaxf(fabsf(mt[r][0]), fabsf(mt[r][1])), fmaxf(fabsf(mt[r][2]), fabsf(mt[r][3])));
      const float av = fmaxf(fmaxf(vt[r][0], vt[r][1]), fmaxf(vt[r][2], vt[r][3]));
      mxm[r] = __reduce_max_sync(kFull, __float_as_uint(am));
      mxv[r] = __reduce_max_sync(kFull, __float_as_uint(av));
    }
    if (lgB >= 8) {
#pragma unroll
      for (int r = 0; r < R; r += 2) {
        mxm[r] = mxm[r + 1] = max(mxm[r], mxm[r + 1]);
        mxv[r] = mxv[r + 1] = max(mxv[r], mxv[r + 1]);
      }
    }
    if (R >= 4 && lgB >= 9) {
      const uint32_t a = max(mxm[0], mxm[R - 2]), b = max(mxv[0], mxv[R - 2]);
#pragma unroll
      for (int r = 0; r < R; ++r) { mxm[r] = a; mxv[r] = b; }
    }

    // ---- per-block constants: lane r works out row r's, then they are broadcast ------------------------
    uint32_t my_m = mxm[0], my_v = mxv[0];
#pragma unroll
    for (int r = 1; r < R; ++r) {
      if ((lane & (R - 1)) == r) { my_m = mxm[r]; my_v = mxv[r]; }
    }
    float my_inv, my_lg;   // my_lg: sqrt2/s for the octave widths, P(s) for 8 and 16 bits
    {
      const float sm = __uint_as_float(my_m);
      const float qmaxf = (float)((1 << (bm - 1)) - 1);
      my_inv = sm < kTiny ? 0.f : __fdiv_rn(qmaxf, sm);
      const float sv = __uint_as_float(my_v);
      if (bv <= 4) my_lg = sv < kTiny ? 0.f : __fmul_rn(__frcp_rn(sv), kSqrt2);
      else my_lg = lg_poly(my_v);
    }
    float s_m[R], inv_m[R];
    LogBlock lb[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const float sm = __uint_as_float(mxm[r]);
      s_m[r] = sm < kTiny ? 0.f : sm;
      inv_m[r] = __shfl_sync(kFull, my_inv, r);
      const float sv = __uint_as_float(mxv[r]);
      const bool zero = sv < kTiny;
      lb[r].s = zero ? 0.f : sv;
      lb[r].c = lb[r].Ps = __shfl_sync(kFull, my_lg, r);
      lb[r].ebase = kMagicBits - (uint32_t)(zero ? kZeroBlockExp : (int)(mxv[r] >> 23));
    }

    // ---- quantize, pack, store; decode the new codes ---------------------------------------------------
    uint8_t* mco = T->mc_out;
    uint8_t* vco = T->vc_out;
    float mq[R][4], vq[R][4];
#define STQ_ENC_M(BW)                                                                                   \
  _Pragma("unroll") for (int r = 0; r < R; ++r)                                                         \
      encode_lin_row<BW>(mco + (size_t)((e_warp + r * kRowElems) >> 3) * BW, lane, mt[r], s_m[r], inv_m[r], mq[r]);
#define STQ_ENC_V(BW)                                                                                   \
  _Pragma("unroll") for (int r = 0; r < R; ++r)                                                         \
      encode_log_row<BW>(vco + (size_t)((e_warp + r * kRowElems) >> 3) * BW, lane, vt[r], lb[r], vq[r]);
    STQ_WIDTH_SWITCH(bm, STQ_ENC_M)
    STQ_WIDTH_SWITCH(bv, STQ_ENC_V)
    if (lane == 0) {
      float* mso = T->ms_out;
      float* vso = T->vs_out;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const uint32_t e_row = e_warp + r * kRowElems;
        if ((e_row & ((1u << lgB) - 1u)) == 0) {
          mso[e_row >> lgB] = s_m[r];
          vso[e_row >> lgB] = lb[r].s;
        }
      }
    }

    // ---- parameter update ------------------------------------------------------------------------------
    const float lrwd = sc.l2_mode ? 0.0f : (float)(sc.lr * (double)wd);
    float* param = T->param + e_warp + 4 * lane;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float out[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float den = __fmaf_rn(sqrt_fast(vq[r][k]), sc.rsqrt_bc2, sc.eps);
        const float upd = __fmul_rn(__fmul_rn(mq[r][k], sc.step_size), rcp_fast(den));
        out[k] = __fadd_rn(th[r][k], -__fmaf_rn(th[r][k], lrwd, upd));
      }
      *reinterpret_cast<float4*>(param + r * kRowElems) = make_float4(out[0], out[1], out[2], out[3]);
    }

    if constexpr (STATS) {
      double dg = (double)st_g, da = (double)st_a, dq = (double)st_q;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        dg += __shfl_down_sync(kFull, dg, o);
        da += __shfl_down_sync(kFull, da, o);
        dq += __shfl_down_sync(kFull, dq, o);
      }
      if (lane == 0) { s_part[warp][0] = dg; s_part[warp][1] = da; s_part[warp][2] = dq; }
      __syncthreads();
      if (tid < 3) {
        double a = 0.0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) a += s_part[w][tid];
        partials[(size_t)tile * 3 + tid] = a;
      }
    }
  }

  // A CTA that gave up raises the flag and waits (bounded again) for the copies it still has in
  // flight, so none lands in shared memory that no longer belongs to it.
  if (failed_at != 0xFFFFFFFFu) {
    if (tid == 0) {
      atomicExch(err_flag, 1);
      for (uint32_t j = failed_at; j < n_my && j < failed_at + kStages; ++j)
        mbar_wait(bar0 + 8 * (j % kStages), (j / kStages) & 1u);
    }
    __syncthreads();
  }
}

template <int GDT, bool STATS>
cudaError_t launch_fast_t(const TensorDesc* table, const uint32_t* tile_map, uint32_t n_fast, const StepConsts& sc,
                          double* partials, int* err_flag, int grid, cudaStream_t stream) {
  static bool attr_set = false;
  auto kern = stq_step_fast_kernel<GDT, STATS>;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int g = (int)(n_fast < (uint32_t)grid ? n_fast : (uint32_t)grid);
  kern<<<g, kThreads, kSmemBytes, stream>>>(table, tile_map, n_fast, sc, partials, err_flag);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_step_fast(int grad_dtype, bool stats, const TensorDesc* table, const uint32_t* tile_map,
                             uint32_t n_fast, const StepConsts& sc, double* partials, int* err_flag, int grid,
                             cudaStream_t stream) {
  if (n_fast == 0) return cudaSuccess;
  if (grad_dtype == 0)
    return stats ? launch_fast_t<0, true>(table, tile_map, n_fast, sc, partials, err_flag, grid, stream)
                 : launch_fast_t<0, false>(table, tile_map, n_fast, sc, partials, err_flag, grid, stream);
  return stats ? launch_fast_t<1, true>(table, tile_map, n_fast, sc, partials, err_flag, grid, stream)
               : launch_fast_t<1, false>(table, tile_map, n_fast, sc, partials, err_flag, grid, stream);
}

int fast_ctas_per_sm() {
  int n = 0;
  auto kern = stq_step_fast_kernel<1, false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return 1;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, kThreads, kSmemBytes) != cudaSuccess) return 1;
  return n > 0 ? n : 1;
}

}  // namespace stq

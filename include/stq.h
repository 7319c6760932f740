/*
 * libstq — mixed-bit quantized AdamW step for NVIDIA B200 (sm_100a).
 *
 * The hot path of STQuant's training step (Algorithm 1, inner loop; Sec. 3.5): every parameter
 * tensor keeps its first moment m (block-wise linear symmetric codes) and second moment v
 * (block-wise logarithmic codes) at its own bit-width; one launch decodes m and v, applies the
 * AdamW update with the re-quantized moments, and writes the new codes at the width assigned for
 * this step.  On decision steps the per-layer gradient sums of Sec. 3.3 ride on the same pass and
 * the host-side transition decision of Sec. 3.4 maps them to new widths.
 *
 * Conventions
 *  - Every pointer in stq_tensor is a DEVICE pointer owned by the caller (host pointers only for
 *    stq_step_host).  param, grad and code buffers must be 16-byte aligned, scale buffers 4-byte.
 *  - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and return without
 *    synchronising, except stq_layer_stats and stq_step_host, which synchronise the stream.
 *  - All arguments are validated on the host before anything is launched.  Return value: 0 on
 *    success, a negative STQ_E_* code otherwise; nothing is launched when an error is returned.
 *    The device code never traps or asserts, and every wait in it is bounded (stq_device_status).
 *  - A handle is bound to one device and is not thread-safe; use one handle per stream.
 *
 * Stored layout (per tensor, per state)
 *  - widths b in {2,3,4,8,16}: codes are an LSB-first little-endian bitstream, element i in bits
 *    [i*b, (i+1)*b); length stq_codes_bytes(numel, b) = ceil(numel*b/8) rounded up to 16 bytes,
 *    padding bits zero.  Scales: one fp32 per block of `block` consecutive elements of the
 *    flattened tensor (last block short), stq_scales_bytes(numel, block) bytes.
 *  - width 32: the codes buffer holds the raw fp32 values (numel*4 rounded up to 16 bytes); the
 *    scale pointers are ignored and may be NULL.
 *  - gradients: fp32, bf16 or fp16, one type per call.
 *  - first moment: code u = q + 2^(b-1), q in [-qmax, qmax], qmax = 2^(b-1)-1, value scale*q/qmax.
 *  - second moment: code u in [0, 2^b-1]; value scale * 2^((u-K)*R/K), K = 2^b-1, R = min(K,30);
 *    code 0 is a floor level, never zero.  A block whose scale is 0 decodes to all zeros.
 *  - second moment, variant STQ_VLOG_PL (per tensor, widths 8 and 16 only; the paper names
 *    logarithmic quantization in Sec. 3.5 without a formula, and this is a second, integer-only
 *    reading of it): log2 is replaced by the piecewise-linear logarithm that the fp32 bit pattern
 *    is.  With D = 30 * 2^23: a value x of a block with scale s has distance
 *    n = min(bits(s) - bits(x), D) and code u = K - floor(n*K/D + 1/2); code u decodes to the
 *    float whose bit pattern is max(bits(s) - floor(j*B/2^S + 1/2), 0), j = K - u,
 *    B = round(D*2^S/K), S = 12 (8 bits) or 20 (16 bits).  Exact at whole octaves below the
 *    maximum; relative error at most 0.7214*30/K octaves.  A state must be read with the variant
 *    it was written with.
 *  - second moment, variant STQ_VLOG_SR (a third reading: stochastic rounding, so that the stored
 *    second moment is an unbiased estimate of the computed one).  Levels: a whole number L = 1, 1, 1,
 *    8, 2048 per octave at widths 2, 3, 4, 8, 16 (g = log2 L), evenly spaced in the mantissa.  With
 *    y = fl(x * fl(fl(1/s) * (1 + 2^-21))) and n = clamp(bits(1.0f) - bits(y), 0, K << (23-g)):
 *    j = min(((n << (9+g)) + U) >> 32, K), code u = K - j, U the element's 32-bit random word;
 *    code u decodes to fl(s * y^), y^ the float with bits(1.0f) - ((K-u) << (23-g)).  Over the random
 *    words E[y^] = y exactly.  mix32(h): h ^= h>>16; h *= 0x85EBCA6B; h ^= h>>13; h *= 0xC2B2AE35;
 *    h ^= h>>16.  h0 = mix32(seed_lo ^ mix32(seed_hi ^ mix32(step_lo ^ mix32(step_hi ^ 0x9E3779B9))))
 *    with seed = stq_hparams.sr_seed and step = stq_hparams.step; key = mix32(stq_tensor.sr_id ^ h0);
 *    U of element e of the row = mix32(e_lo ^ mix32(key + e_hi)).  stq_repack has no step to draw
 *    from and rounds to nearest (U = 2^31).  Re-quantization is not idempotent in this variant.
 *  - second moment, variant STQ_VLOG_TS (a fourth reading: two scales per block).  The scale buffer
 *    holds two floats per block, {hi, lo}: hi = max x, lo = max(min x, hi * 2^-30); size
 *    stq_v_scales_bytes().  With d(x) the split logarithm of x/hi as in the main code and
 *    W = min(-d(lo), 30): u = clamp(K + rne(clamp(d(x), -W, 0) * fl(K/W)), 0, K); u = 0 decodes to
 *    lo, otherwise fl(hi * ex(fl((u-K) * fl(W/K)))): both end points exact, error at most W/(2K)
 *    octaves.  W = 0 (all elements equal): every code is K.
 */
#ifndef STQ_H_
#define STQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct stq_handle stq_handle;
typedef struct stq_policy stq_policy;

enum {
  STQ_OK = 0,
  STQ_E_NULL = -1,      /* a required pointer is NULL                                         */
  STQ_E_BITS = -2,      /* a width outside {2,3,4,8,16,32}                                    */
  STQ_E_BLOCK = -3,     /* block is not a power of two in 32..1024                            */
  STQ_E_ALIGN = -4,     /* a buffer is not aligned as required                                */
  STQ_E_ALIAS = -5,     /* in/out buffers overlap in a way the step cannot honour             */
  STQ_E_NUMEL = -6,     /* numel == 0, or the table is empty or too large                     */
  STQ_E_CUDA = -7,      /* a CUDA runtime call failed (see stq_last_cuda_error)               */
  STQ_E_WORKSPACE = -8, /* the library could not grow its own workspace                       */
  STQ_E_ARG = -9,       /* an invalid scalar argument (step < 1, unknown dtype or flag, ...)  */
  STQ_E_STATE = -10,    /* call order: no statistics pending for stq_layer_stats              */
  STQ_E_TIMEOUT = -11,  /* a bounded wait inside a kernel ran out (stq_device_status)         */
  STQ_E_TOO_LARGE = -12 /* the tensor exceeds the fixed capacity of an entry point that does  */
                        /* not allocate (stq_grad_stats_static)                               */
};

enum { STQ_GRAD_F32 = 0, STQ_GRAD_BF16 = 1, STQ_GRAD_F16 = 2 };

/* type of the optional low-precision copy of the updated parameters (stq_tensor.param_lp) */
enum { STQ_LP_NONE = 0, STQ_LP_BF16 = 1, STQ_LP_F16 = 2 };

/* quantizer of the second moment (stq_tensor.v_log); see "Stored layout".  POLY and PL differ at widths 8 and
 * 16 only; SR and TS are codes of their own at every width and run in the generic kernel. */
enum { STQ_VLOG_POLY = 0, STQ_VLOG_PL = 1, STQ_VLOG_SR = 2, STQ_VLOG_TS = 3 };

/* flags of stq_step */
enum { STQ_WITH_STATS = 1u };

/* The step kernels work on tiles of this many consecutive elements of one tensor.  A tensor whose numel is a
 * multiple of it (with packed states and a block of 128 or 256) is served by the main kernel alone; the ragged last
 * tile of any other tensor goes to the generic kernel, which costs a step one more launch.  A caller that owns its
 * buffers can avoid that by padding every buffer of a tensor with zeros to a whole number of tiles and passing the
 * padded numel: zero gradients keep the padding at zero, it adds nothing to the statistics' sums (only the element
 * count reported by stq_layer_stats is then the padded one) and leaves the real elements' blocks as they are
 * (except under STQ_VLOG_TS, whose block minimum the padding inside a last, partly real block would change). */
#define STQ_TILE_ELEMS 4096

/* One row per parameter tensor (a "layer" of the paper is one tensor). */
typedef struct stq_tensor {
  float* param;              /* fp32 master weights, numel elements, updated in place          */
  const void* grad;          /* numel gradients, fp32 or bf16 (stq_hparams.grad_dtype)         */
  const void* m_codes_in;    /* stored first moment: codes at width bits_m                     */
  const float* m_scales_in;  /*                      block scales (ignored when bits_m == 32)  */
  const void* v_codes_in;    /* stored second moment: codes at width bits_v                    */
  const float* v_scales_in;
  void* m_codes_out;         /* written at width bits_m_out; may be the same pointer as        */
  float* m_scales_out;       /* m_codes_in only if bits_m_out == bits_m (no partial overlap);  */
  void* v_codes_out;         /* scales_out may equal scales_in                                 */
  float* v_scales_out;
  uint64_t numel;
  uint32_t block;            /* quantization block: a power of two, 32..1024 (128 and 256 run   */
                             /* in the main kernel, the others in the generic one)             */
  uint8_t bits_m, bits_v;          /* widths stored now                                        */
  uint8_t bits_m_out, bits_v_out;  /* widths to write                                          */
  float weight_decay;        /* per-tensor lambda                                              */
  uint32_t lp_dtype;         /* STQ_LP_*: type of param_lp (STQ_LP_NONE: no copy)              */
  void* param_lp;            /* optional: numel elements that receive the updated parameters   */
                             /* rounded (nearest-even) to lp_dtype, the model's working copy   */
                             /* in mixed-precision training; 8-byte aligned; written by         */
                             /* stq_step only                                                  */
  uint32_t v_log;            /* STQ_VLOG_*: how the second moment is coded, on the way in and  */
                             /* on the way out                                                 */
  uint32_t sr_id;            /* STQ_VLOG_SR: identifies this tensor in the random stream (use   */
                             /* its index in the model); 0 otherwise                           */
} stq_tensor;

typedef struct stq_hparams {
  double lr, beta1, beta2, eps;
  int64_t step;          /* t >= 1: the step being taken (bias correction 1 - beta^t)          */
  int32_t decoupled_wd;  /* 1: AdamW as in Algorithm 1; 0: weight decay added to the gradient  */
  int32_t grad_dtype;    /* STQ_GRAD_F32, STQ_GRAD_BF16 or STQ_GRAD_F16                        */
  /* Loss-scaled training (the paper trains in FP16): both are DEVICE pointers to one float, or NULL. */
  const float* inv_grad_scale; /* every gradient is multiplied by *inv_grad_scale (1 / loss scale)   */
                               /* before anything else (statistics included)                         */
  const float* found_inf;      /* if *found_inf != 0 the step is skipped: no buffer is touched, and   */
                               /* statistics requested with the step are not produced (the next      */
                               /* stq_layer_stats returns STQ_E_STATE; the value is read when the     */
                               /* step runs, so the caller may reuse the flag afterwards)            */
  /* Step count and learning rate kept on the DEVICE (both optional, NULL = use `step` and `lr` above):  */
  /* a step captured into a CUDA graph then advances with the caller's counter instead of repeating     */
  /* the captured t.  The bias corrections 1 - beta^t are formed on the device in double precision.     */
  const int64_t* step_dev;     /* device pointer to t >= 1 (values below 1 are read as 1)              */
  const float* lr_dev;         /* device pointer to the learning rate                                  */
  uint64_t sr_seed;            /* seed of the random words of STQ_VLOG_SR tensors (with `step`; not     */
                               /* available together with step_dev)                                    */
} stq_hparams;

/* Handle: device copy of the tensor table, tile map and statistics workspace.
 * stq_create makes `device` current for the call and allocates nothing large; workspaces grow on
 * first use (cudaMalloc) and are freed by stq_destroy. */
int stq_create(stq_handle** out, int device);
int stq_destroy(stq_handle* h);

/* Buffer sizes of the stored layout described above. */
size_t stq_codes_bytes(uint64_t numel, int bits);
size_t stq_scales_bytes(uint64_t numel, uint32_t block);
/* Scale buffer of a second moment coded with variant v_log: two floats per block for STQ_VLOG_TS. */
size_t stq_v_scales_bytes(uint64_t numel, uint32_t block, uint32_t v_log);

/* Algorithm 1, initialisation: m = v = 0.  Writes the canonical zero state (first-moment codes
 * 2^(b-1), second-moment codes 0, all scales 0) into the *_out buffers at bits_m_out/bits_v_out.
 * param, grad and the *_in fields are ignored. */
int stq_init_state(stq_handle* h, const stq_tensor* tensors, int L, void* stream);

/* Algorithm 1, inner loop, for all L tensors in one pass:
 *   m_t = beta1*m + (1-beta1)*g,  v_t = beta2*v + (1-beta2)*g^2      (states decoded from *_in)
 *   codes/scales_out = Quantize(m_t, linear), Quantize(v_t, log)      (at bits_*_out)
 *   param = param*(1 - lr*wd) - lr * (mq/(1-beta1^t)) / (sqrt(vq/(1-beta2^t)) + eps)
 * where mq, vq are the values the new codes decode to.  With STQ_WITH_STATS the per-tensor sums
 * sum g, sum |g|, sum g^2 (Eq. 2, 3, 8) are accumulated in the same pass; fetch them with
 * stq_layer_stats.
 * Stream capture: the first call with a given table validates it and uploads it (host work that
 * may synchronise); a later call with the byte-identical table only enqueues work on `stream` and on
 * an internal side stream forked from and joined back into it, so it can be captured into a CUDA
 * graph.  The scalars derived from `hp` (bias corrections, learning rate) are launch parameters:
 * a replay repeats the captured step t. */
int stq_step(stq_handle* h, const stq_tensor* tensors, int L, const stq_hparams* hp, unsigned flags,
             void* stream);

/* Gradient statistics alone (Algorithm 1 computes them before the update): reads only grad and
 * numel of each row.  Fetch with stq_layer_stats. */
int stq_grad_stats(stq_handle* h, const stq_tensor* tensors, int L, int grad_dtype, void* stream);

/* Finishes the reduction started by the last stq_step(STQ_WITH_STATS) or stq_grad_stats on this
 * handle and copies it to HOST memory: out[l] = {sum g, sum |g|, sum g^2, numel} for l < L.
 * Synchronises `stream`.  The reduction order is fixed, so results are run-to-run identical.
 * Call order: the sums stay pending while the handle keeps seeing the table they were taken with
 * (further steps over the byte-identical table are fine).  Any call with another table on the same
 * handle (stq_repack, stq_init_state, a step with other pointers or widths) drops them, and so does a
 * step that found_inf skipped: this call then returns STQ_E_STATE and writes nothing.  Fetch the sums
 * before re-packing or changing widths. */
int stq_layer_stats(stq_handle* h, double* out, int L, void* stream);

/* The same sums as stq_grad_stats + stq_layer_stats for ONE gradient tensor, for callers that must
 * not trigger a device allocation (the paper has no counterpart: this is plumbing).  Typical
 * cases: the training process has already given all free device memory to its own caching
 * allocator, so a cudaMalloc from a library can fail or stall the device in mid-step; or the
 * caller runs under a fixed memory budget.  This call needs no handle, calls no allocating routine
 * and keeps its scratch (one partial sum per 4096 elements) in a static device array inside the
 * library: 393,472 bytes that every GPU loading the library holds until the process exits.
 *   - numel may be at most STQ_STATIC_STATS_MAX_NUMEL; larger tensors are rejected with
 *     STQ_E_TOO_LARGE and nothing is launched (split the tensor and add the sums).
 *   - grad: device pointer, 16-byte aligned, fp32 or bf16.  out: DEVICE pointer to 4 doubles
 *     {sum g, sum |g|, sum g^2, numel}, written on `stream`; the call does not synchronise.
 *   - `device` is made current.  The first call on a device also looks up the device address of
 *     the scratch array; make that first call before any stream capture begins.
 *   - All calls on a device share the scratch array, which keeps the previous call's contents;
 *     the one word that must start at zero is cleared on `stream` by every call.  Calls that
 *     overlap on the GPU (different streams without ordering between them) race on the scratch:
 *     keep them ordered. */
#define STQ_STATIC_STATS_MAX_NUMEL (64ull * 1024 * 1024)
int stq_grad_stats_static(int device, const void* grad, uint64_t numel, int grad_dtype, double* out, void* stream);

/* Width transition without an optimizer step (implied by the per-step widths b_{l,t} of
 * Sec. 3.1): codes_out = Quantize_{bits_out}(Decode_{bits}(codes_in)) for both states; block
 * scales are recomputed and come out unchanged for quantized sources.  bits 32 on either side
 * turns this into a plain quantize / decode of raw fp32 states.  param and grad are ignored. */
int stq_repack(stq_handle* h, const stq_tensor* tensors, int L, void* stream);

/* stq_step with every pointer in `tensors` a HOST pointer: the library stages the buffers through
 * a device arena it owns (grown on demand), copies param/grad/codes/scales in, runs the step,
 * copies param/codes/scales back and synchronises the device.  Chunks of consecutive tensors
 * (~256 MB) are pipelined over three internal streams, so with pinned host buffers the copies in,
 * the kernels and the copies out overlap (a step with STQ_WITH_STATS runs as one chunk).
 * Layout matters for speed, not for the result: where the buffers of one kind (param, grad, the
 * codes or the scales of one state) of consecutive tensors lie back to back in host memory, with
 * gaps of at most 4096 bytes between them, a chunk moves them as ONE copy per kind and direction
 * (the gap bytes are read and written back unchanged, so they must belong to the caller and stay
 * untouched during the call); buffers allocated one by one are copied one by one, which costs
 * about a third of the throughput on tables of hundreds of tensors.
 * bytes_h2d / bytes_d2h (optional) receive the bytes copied. */
int stq_step_host(stq_handle* h, const stq_tensor* tensors, int L, const stq_hparams* hp,
                  unsigned flags, uint64_t* bytes_h2d, uint64_t* bytes_d2h);

/* Synchronises `stream` and reports whether any kernel launched through this handle gave up on a
 * bounded wait (its asynchronous copies did not complete in ~2 s): STQ_E_TIMEOUT, else STQ_OK.
 * The device never spins without a limit; after a time-out the outputs of that launch are
 * undefined and the handle should be destroyed. */
int stq_device_status(stq_handle* h, void* stream);

/* Exercises the time-out path without stalling anything: launches a one-warp kernel that waits, with
 * a ~0.1 ms limit, on a barrier nothing completes, and raises the handle's error flag exactly as a
 * stalled copy in the step kernel would.  Afterwards stq_device_status returns STQ_E_TIMEOUT for this
 * handle (the flag is sticky); the CUDA context stays usable.  For tests of the failure reporting. */
int stq_selftest_wait_timeout(stq_handle* h, void* stream);

/* Kernel launches issued through this handle so far. */
uint64_t stq_launch_count(const stq_handle* h);
/* Persistent grid the step kernel uses on this device (CTAs), and the device's SM count. */
int stq_grid_size(const stq_handle* h);
int stq_sm_count(const stq_handle* h);

/* ---- transition decision (host only; Sec. 3.3-3.4, Algorithm 1 decision branch) -------------- */
typedef struct stq_policy_cfg {
  double alpha;         /* EMA factor of the three global running statistics                  */
  double tau;           /* decay period of the annealing factor S_t = 1 + sech(t/tau) (Eq. 7) */
  double eps_stat;      /* the small constant in r_l and in the score denominators            */
  int64_t interval;     /* U: decide when t mod U == 0 or t < 5                               */
  int32_t cv_of_signed; /* 0: sigma(|g|)/mu(|g|) (Eq. 3); 1: sigma(g)/E|g| (Algorithm 1 text)  */
  int32_t reserved;
} stq_policy_cfg;

int stq_policy_create(stq_policy** out, const stq_policy_cfg* cfg);
int stq_policy_destroy(stq_policy* p);
/* 1 if Algorithm 1 takes the decision branch at step t. */
int stq_policy_is_decision_step(const stq_policy* p, int64_t t);
/* One decision, O(L): updates the running averages from stats[L][4] (as written by
 * stq_layer_stats), then score_l = 7.2 + log2 ratios (Sec. 3.4) and bits_out[l] = Map(score_l)
 * in {4, 8, 16, 32} with thresholds 6.8 / 12 / 24.  score_out may be NULL. */
int stq_decide(stq_policy* p, const double* stats, int L, int64_t t, uint8_t* bits_out,
               double* score_out);
/* Running averages {n, r, v} for checkpointing. */
int stq_policy_get_state(const stq_policy* p, double out[3]);
int stq_policy_set_state(stq_policy* p, const double in[3]);

const char* stq_strerror(int code);
/* Text of the last CUDA error seen by this handle ("" if none). */
const char* stq_last_cuda_error(const stq_handle* h);

#ifdef __cplusplus
}
#endif
#endif /* STQ_H_ */

// Internal interface between the C-ABI host layer (stq_api.cu) and the kernels (stq_kernels.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace stq {

constexpr int kThreads = 256;    // 8 warps per CTA
constexpr int kRowElems = 128;   // one row: lane l holds elements 4l .. 4l+3
constexpr int kRowsPerWarp = 4;  // a warp owns this many consecutive rows of a tile
constexpr int kTile = (kThreads / 32) * kRowsPerWarp * kRowElems;   // elements per tile; a tile lies inside one tensor
constexpr int kMinBlock = 32;                                       // a lane's four elements never straddle blocks
constexpr int kMaxBlock = 2 * kRowsPerWarp * kRowElems;             // a quantization block spans at most two warps of a tile
constexpr int kFastCtasPerSm = 2;   // resident CTAs per SM of the main step kernel
constexpr int kFastStages = 2;      // depth of its shared-memory ring
constexpr int kFastRowsPerPass = 2; // rows a warp handles per pass over its kRowsPerWarp rows (see the kernel)
constexpr int kFastMaxBlock = kFastRowsPerPass * kRowElems;   // larger blocks take the generic path

// Device-side row of the tensor table.
struct TensorDesc {
  float* param;
  const void* grad;
  const uint8_t* mc_in;
  const float* ms_in;
  const uint8_t* vc_in;
  const float* vs_in;
  uint8_t* mc_out;
  float* ms_out;
  uint8_t* vc_out;
  float* vs_out;
  unsigned long long numel;
  unsigned int tile0;       // first "fast" tile (full tile, same width in and out) of this tensor
  unsigned int nfast;       // number of fast tiles; they cover elements [0, nfast * kTile)
  unsigned int tile0s;      // first tile of the rest (ragged tail, or the whole tensor if it is not fast)
  unsigned int nslow;
  unsigned int seg0;        // first statistics segment (kStatSegTiles tiles each) of this tensor
  unsigned int block;       // power of two, 32 .. 1024
  unsigned char bm_in, bv_in, bm_out, bv_out;
  float wd;                 // fp32(lambda)
  unsigned int lp_dtype;    // 0: none, 1: bf16, 2: fp16
  unsigned int v_mode;      // code of the second moment: 0 polynomial logarithm, 1 piecewise-linear one (differs at
                            // widths 8 and 16), 2 stochastic rounding, 3 two scales per block (generic kernel only)
  unsigned int sr_id;       // identifies the tensor in the random stream of the stochastic-rounding code
  void* param_lp;           // low-precision copy of the updated parameters, or nullptr
};

// Per-launch scalars of the AdamW update.
struct StepConsts {
  float b1, c1, b2, c2;     // fp32(beta), fp32(1-beta): the bit-exact moment recursion
  float step_size;          // lr / (1 - beta1^t)
  float rsqrt_bc2;          // 1 / sqrt(1 - beta2^t)
  float eps;
  unsigned int sr_h;        // stochastic rounding: the word mixed from (seed, step); the key of a tensor is mix32(sr_id ^ sr_h)
  float one;                // 1.0f as a run-time value (see the packed arithmetic of the main step kernel)
  int l2_mode;              // 1: g += wd*theta before the moments, no decoupled decay
  double lr;                // decoupled decay factor is fp32(1 - lr*wd), formed per tile
  const float* inv_scale;   // device: gradients are multiplied by *inv_scale first (nullptr: no)
  const float* found_inf;   // device: a non-zero value skips the whole step (nullptr: never)
  const float* dev_scalars; // device: {step_size, rsqrt_bc2, lr} written by the scalars kernel for this launch
                            // (nullptr: the three values above are the ones to use)
};

// Derives the step's scalars from a step count (and optionally a learning rate) held on the device:
// out = {lr / (1 - beta1^t), 1 / sqrt(1 - beta2^t), lr}, in double precision, one thread.
cudaError_t launch_step_scalars(const long long* step_dev, const float* lr_dev, double lr_host, double beta1,
                                double beta2, float* out, cudaStream_t stream);

// Records whether a call that is to carry statistics will produce them: *valid = 1 unless *found_inf (device,
// may be nullptr) is non-zero, in which case the step kernels return without writing a partial sum.
cudaError_t launch_stats_valid(const float* found_inf, int* valid, cudaStream_t stream);

enum Mode { kStep = 0, kRepack = 1, kInit = 2, kStatsOnly = 3 };

// Launches the tile range [tile_begin, tile_end) of the table.  `wide` selects the variant that
// can read/write 32-bit (raw fp32) states, `variants` the one that knows the second-moment codes only the
// generic kernel serves.  partials: 3 doubles per warp and tile, or nullptr.
cudaError_t launch_tiles(Mode mode, bool wide, bool variants, int grad_dtype, bool stats, const TensorDesc* table,
                         const uint32_t* tile_map, uint32_t tile_begin, uint32_t tile_end,
                         const StepConsts& sc, double* partials, int grid, cudaStream_t stream);

// Work list of the main step kernel: the fast tiles [0, n_fast) of the tile order, cut into groups
// of equal body (width pair, variant of the v code).  Lives in device memory; the counters are zeroed before every launch.
constexpr int kFastMaxGroups = 64;     // 5 widths of m x (5 widths of v + 2 variants at 8 and 16 bits) = 35 bodies
constexpr int kFastMaxGrid = 4096;
constexpr uint32_t kFastChunk = 2;     // tiles handed out per counter increment (one for small launches); measured:
                                       // 2-3 beat 1 and 8 by 1-4 % on the small and medium configurations (shorter tail
                                       // when a group runs dry), no difference on the largest
struct FastSched {
  uint32_t ctr[kFastMaxGroups];            // chunks handed out so far, per group (zero between launches: see `done`)
  uint32_t done;                           // CTAs that have left their hand-out loop; the last one zeroes the counters
  uint32_t ng;                             // number of groups
  uint32_t chunk;                          // tiles per counter increment for this launch
  uint32_t grp_begin[kFastMaxGroups + 1];  // tile range of group g: [grp_begin[g], grp_begin[g+1])
  uint16_t cta_group[kFastMaxGrid];        // group a CTA starts in
};

// The main step kernel (stq_step_fast.cuh) with `grid` CTAs.  err_flag is set to 1 if a bounded wait
// inside the kernel ran out.
// amp: some tensor wants a low-precision copy, or the gradients are loss-scaled.
// list: 0 the fused bodies of the default and "pl" codes, 1 the fused bodies of the "sr" and "ts" codes, 2 the
// tiles of tensors whose widths change inside the step (each its own work list and instantiation).
cudaError_t launch_step_fast(int grad_dtype, bool stats, bool amp, int list, const TensorDesc* table,
                             const uint32_t* tile_map, FastSched* sched, const StepConsts& sc, double* partials,
                             int* err_flag, int grid, cudaStream_t stream);
// (the launches of work lists 1 and 2, each instantiated in a translation unit of its own)
cudaError_t launch_step_fast_variants(int grad_dtype, const TensorDesc* table, const uint32_t* tile_map, FastSched* sched,
                                      const StepConsts& sc, double* partials, int* err_flag, int grid, cudaStream_t stream);
cudaError_t launch_step_fast_split(int grad_dtype, const TensorDesc* table, const uint32_t* tile_map, FastSched* sched,
                                   const StepConsts& sc, double* partials, int* err_flag, int grid, cudaStream_t stream);
int fast_ctas_per_sm();
// Launches the time-out self-test (see stq_step_fast.cu): sets *err_flag after a ~0.1 ms bounded wait.
cudaError_t launch_wait_timeout_selftest(int* err_flag, cudaStream_t stream);

// Second stage of the statistics.  A tensor's tiles (fast range, then the rest) are cut into
// segments of kStatSegTiles tiles; seg_map[s] is the tensor of segment s.  First every segment is
// summed (seg_sums: 3 doubles per segment), then every tensor adds its segments:
// out[l] = {sum g, sum |g|, sum g^2, numel}.  All orders are fixed, so results are reproducible.
constexpr int kStatSegTiles = 32;
cudaError_t launch_stats_finish(const TensorDesc* table, int L, const uint32_t* seg_map, uint32_t n_seg,
                                const double* partials, double* seg_sums, double* out, cudaStream_t stream);

// Resident CTAs per SM of the step kernel (occupancy query), for sizing the persistent grid.
int step_ctas_per_sm();

}  // namespace stq

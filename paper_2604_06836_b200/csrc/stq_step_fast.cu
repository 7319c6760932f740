// The main launches of the step kernel (stq_step_fast.cuh): the fused bodies of the default and "pl" codes.  The
// fused bodies of the "sr" and "ts" codes are instantiated in stq_step_variants.cu, the runtime-width body of tensors
// that change width inside the step in stq_step_split.cu.
#include "stq_step_fast.cuh"

namespace stq {
namespace {

// Self-test of the time-out path: one warp waits, with a short limit, on a barrier phase that nothing
// will ever complete, finds the limit, raises the flag and returns.  The same code path a stalled
// copy would take in the step kernel, without stalling anything.
__global__ void stq_wait_timeout_selftest_kernel(int* __restrict__ err_flag, long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool done = mbar_wait(b, 0u, limit_cycles);
  if (!done && threadIdx.x == 0) atomicExch(err_flag, 1);
}


}  // namespace

cudaError_t launch_step_fast(int grad_dtype, bool stats, bool amp, int list, const TensorDesc* table,
                             const uint32_t* tile_map, FastSched* sched, const StepConsts& sc, double* partials,
                             int* err_flag, int grid, cudaStream_t stream) {
  double* p = stats ? partials : nullptr;
#define STQ_LAUNCH(G, A, S) return launch_fast_t<G, A, S>(table, tile_map, sched, sc, p, err_flag, grid, stream)
#define STQ_LAUNCH_G(A, S)              \
  switch (grad_dtype) {                 \
    case 0: STQ_LAUNCH(0, A, S);        \
    case 1: STQ_LAUNCH(1, A, S);        \
    default: STQ_LAUNCH(2, A, S);       \
  }
  if (list == 2) return launch_step_fast_split(grad_dtype, table, tile_map, sched, sc, p, err_flag, grid, stream);
  if (list == 1) return launch_step_fast_variants(grad_dtype, table, tile_map, sched, sc, p, err_flag, grid, stream);
  if (amp) {
    STQ_LAUNCH_G(true, 0)
  }
  STQ_LAUNCH_G(false, 0)
#undef STQ_LAUNCH_G
#undef STQ_LAUNCH
}

cudaError_t launch_wait_timeout_selftest(int* err_flag, cudaStream_t stream) {
  stq_wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(err_flag, 200000ll);   // ~0.1 ms
  return cudaGetLastError();
}

int fast_ctas_per_sm() {
  int n = 0;
  auto kern = stq_step_fast_kernel<1, false, 0>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return 1;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, kFastThreads, kSmemBytes) != cudaSuccess) return 1;
  return n > 0 ? n : 1;
}

}  // namespace stq

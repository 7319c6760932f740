// The step kernel over the tiles of tensors that change width inside the step (work list 2: one runtime-width body).
#include "stq_step_fast.cuh"

namespace stq {

cudaError_t launch_step_fast_split(int grad_dtype, const TensorDesc* table, const uint32_t* tile_map, FastSched* sched,
                                   const StepConsts& sc, double* partials, int* err_flag, int grid, cudaStream_t stream) {
  // (the mixed-precision extras cost these bodies nothing measurable: one instantiation serves both)
  switch (grad_dtype) {
    case 0: return launch_fast_t<0, true, 2>(table, tile_map, sched, sc, partials, err_flag, grid, stream);
    case 1: return launch_fast_t<1, true, 2>(table, tile_map, sched, sc, partials, err_flag, grid, stream);
    default: return launch_fast_t<2, true, 2>(table, tile_map, sched, sc, partials, err_flag, grid, stream);
  }
}

}  // namespace stq

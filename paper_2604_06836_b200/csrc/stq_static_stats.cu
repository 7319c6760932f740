// stq_grad_stats_static: the per-layer gradient sums without any allocation.
//
// Some callers cannot let a library allocate device memory.  A training process usually hands
// almost all free device memory to its own caching allocator during warm-up; a cudaMalloc issued
// later by a library may then fail although the framework still holds plenty of free blocks, and
// even when it succeeds it synchronises the whole device in the middle of a step.  Code that runs
// under a fixed memory budget, or inside a region where the framework forbids allocation, is in
// the same position.  For those callers this entry point keeps its scratch memory in a
// file-scope __device__ array that is part of the library image: every GPU that loads the library
// holds those bytes until the process exits, nothing is allocated or freed at run time, and the
// price is a fixed upper limit on the tensor size.
//
// The scratch array is shared by all calls on a device and keeps whatever the last call left in
// it.  The only word that has to start at zero (the arrival counter) is cleared on the stream at
// the start of every call.  Two calls that overlap on the GPU (different streams, or different
// host threads without ordering) would use the same scratch at once and race: keep calls on one
// device ordered.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/stq.h"

namespace {

constexpr int kTileElems = 4096;                        // elements reduced by one CTA
constexpr int kThreadsStatic = 256;
constexpr unsigned long long kMaxNumel = STQ_STATIC_STATS_MAX_NUMEL;
constexpr int kMaxTiles = (int)(kMaxNumel / kTileElems);
constexpr int kHeaderDoubles = 32;                      // 256 bytes: the arrival counter lives here

// [0, 256): header (arrival counter), then three doubles per tile.  393,472 bytes per GPU.
static __device__ __align__(256) double g_static_scratch[kHeaderDoubles + 3 * kMaxTiles];

__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }

template <int GDT>
__global__ void __launch_bounds__(kThreadsStatic)
stq_static_stats_kernel(const void* __restrict__ grad, unsigned long long numel, double* __restrict__ scratch,
                        double* __restrict__ out) {
  __shared__ double sh[kThreadsStatic][3];
  __shared__ bool is_last;
  const int tid = threadIdx.x;
  const unsigned long long base = (unsigned long long)blockIdx.x * kTileElems;

  // this CTA's tile: every thread takes four groups of four consecutive elements
  float sg = 0.f, sa = 0.f, sq = 0.f;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const unsigned long long e = base + (unsigned long long)k * 1024 + 4 * tid;
    float g[4] = {0.f, 0.f, 0.f, 0.f};
    if (e + 4 <= numel) {
      if constexpr (GDT == 0) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(grad) + e));
        g[0] = v.x; g[1] = v.y; g[2] = v.z; g[3] = v.w;
      } else {
        const uint2 v = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(grad) + e));
        g[0] = __uint_as_float(v.x << 16); g[1] = __uint_as_float(v.x & 0xFFFF0000u);
        g[2] = __uint_as_float(v.y << 16); g[3] = __uint_as_float(v.y & 0xFFFF0000u);
      }
    } else {
      for (int j = 0; j < 4; ++j) {
        if (e + j < numel) {
          if constexpr (GDT == 0) g[j] = __ldg(reinterpret_cast<const float*>(grad) + e + j);
          else g[j] = bf16_bits_to_float(__ldg(reinterpret_cast<const uint16_t*>(grad) + e + j));
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      sg += g[j];
      sa += fabsf(g[j]);
      sq = fmaf(g[j], g[j], sq);
    }
  }
  sh[tid][0] = (double)sg; sh[tid][1] = (double)sa; sh[tid][2] = (double)sq;
  __syncthreads();
  for (int s = kThreadsStatic / 2; s > 0; s >>= 1) {
    if (tid < s) {
#pragma unroll
      for (int k = 0; k < 3; ++k) sh[tid][k] += sh[tid + s][k];
    }
    __syncthreads();
  }

  // publish the tile's partial, then take a ticket: the CTA that arrives last finishes the job
  double* part = scratch + kHeaderDoubles;
  unsigned int* counter = reinterpret_cast<unsigned int*>(scratch);
  if (tid < 3) part[(size_t)blockIdx.x * 3 + tid] = sh[0][tid];
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    __threadfence();   // the publishing thread itself orders the three stores (seen through the barrier) before its ticket
    is_last = (atomicAdd(counter, 1u) == gridDim.x - 1);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();

  // fixed-order sum of all partials (the same order whatever CTA happens to be last)
  double a[3] = {0.0, 0.0, 0.0};
  for (unsigned int t = tid; t < gridDim.x; t += kThreadsStatic) {
#pragma unroll
    for (int k = 0; k < 3; ++k) a[k] += __ldcg(part + (size_t)t * 3 + k);
  }
#pragma unroll
  for (int k = 0; k < 3; ++k) sh[tid][k] = a[k];
  __syncthreads();
  for (int s = kThreadsStatic / 2; s > 0; s >>= 1) {
    if (tid < s) {
#pragma unroll
      for (int k = 0; k < 3; ++k) sh[tid][k] += sh[tid + s][k];
    }
    __syncthreads();
  }
  if (tid < 3) out[tid] = sh[0][tid];
  if (tid == 3) out[3] = (double)numel;
}

// Device address of the scratch array, resolved once per device.  In host code the array's name
// is only a stand-in for the symbol, not an address a kernel could use.
constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
double* g_scratch_addr[kMaxDevices] = {nullptr};

int scratch_for_device(int device, double** out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[device] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return STQ_E_CUDA;
    g_scratch_addr[device] = static_cast<double*>(p);
  }
  *out = g_scratch_addr[device];
  return STQ_OK;
}

}  // namespace

extern "C" int stq_grad_stats_static(int device, const void* grad, uint64_t numel, int grad_dtype, double* out,
                                     void* stream) {
  if (!grad || !out) return STQ_E_NULL;
  if (grad_dtype != STQ_GRAD_F32 && grad_dtype != STQ_GRAD_BF16) return STQ_E_ARG;
  if (numel == 0) return STQ_E_NUMEL;
  if (numel > kMaxNumel) return STQ_E_TOO_LARGE;   // the static scratch holds one partial per 4096 elements
  if ((reinterpret_cast<uintptr_t>(grad) & 15u) != 0 || (reinterpret_cast<uintptr_t>(out) & 7u) != 0) return STQ_E_ALIGN;
  if (device < 0 || device >= kMaxDevices) return STQ_E_ARG;
  if (cudaSetDevice(device) != cudaSuccess) return STQ_E_CUDA;
  double* scratch = nullptr;
  int rc = scratch_for_device(device, &scratch);
  if (rc != STQ_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the arrival counter must start at zero; everything else in the scratch is overwritten before it is read
  if (cudaMemsetAsync(scratch, 0, kHeaderDoubles * sizeof(double), s) != cudaSuccess) return STQ_E_CUDA;
  const unsigned int tiles = (unsigned int)((numel + kTileElems - 1) / kTileElems);
  if (grad_dtype == STQ_GRAD_F32)
    stq_static_stats_kernel<0><<<tiles, kThreadsStatic, 0, s>>>(grad, numel, scratch, out);
  else
    stq_static_stats_kernel<1><<<tiles, kThreadsStatic, 0, s>>>(grad, numel, scratch, out);
  return cudaGetLastError() == cudaSuccess ? STQ_OK : STQ_E_CUDA;
}

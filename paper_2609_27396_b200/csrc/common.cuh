// Shared host/device helpers of the dpara kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/dpara.h"

namespace dpara {

constexpr int kNumSM = 148;  // B200: 2 dies x 74 SMs; grids are sized in multiples of this where it matters

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Launch-error check used by the host entry points: returns DPARA_ERR_CUDA from the caller.
#define DPARA_CHECK_LAUNCH()                                   \
  do {                                                         \
    cudaError_t e_ = cudaGetLastError();                       \
    if (e_ != cudaSuccess) return DPARA_ERR_CUDA;              \
  } while (0)

// Programmatic dependent launch.  Every kernel of this library runs pdl_wait() (blocks until the kernels before it have
// completed and their writes are visible) BEFORE it reads or writes any global memory, then pdl_launch_dependents() (the
// next kernel on the stream may be set up and its CTAs made resident as SMs free up); launched through launch_pdl the
// kernel's launch latency and set-up then overlap its predecessor.  Wait first, trigger second: a dependent is only ever
// released by a kernel whose own predecessors are complete, so a dependent that reads some of its inputs before its own
// wait (the early-start form of verify/select) can race with nothing older than its immediate predecessor.  Without the
// launch attribute both instructions do nothing.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Process-wide count of kernels this library has launched (evidence for benchmarks; relaxed atomic).
void count_launches(int n);

}  // namespace dpara

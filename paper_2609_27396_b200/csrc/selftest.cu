// Self-test of the bounded device-side wait that every kernel of this library uses for its mbarriers:
// one CTA waits on a barrier that nothing ever arrives at; the wait must give up after its time limit,
// report DPARA_STATUS_TIMEOUT through the status word and let the kernel end normally (no trap, no hang),
// leaving the context usable.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dpara {

__global__ void bounded_wait_selftest_kernel(int32_t *status_word, uint64_t limit_ns, unsigned long long *waited_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  const uint64_t t0 = ptx::global_timer_ns();
  const bool ok = ptx::mbar_wait_limit(&bar, 0, &abort_flag, limit_ns);  // never armed: must time out
  __syncthreads();
  if (threadIdx.x == 0) {
    if (waited_ns) *waited_ns = ptx::global_timer_ns() - t0;
    if (!ok && status_word) atomicOr(reinterpret_cast<unsigned int *>(status_word), DPARA_STATUS_TIMEOUT);
  }
}

}  // namespace dpara

extern "C" dpara_status dpara_selftest_bounded_wait(int32_t *status_word, uint32_t limit_us, uint64_t *waited_ns, void *stream) {
  if (!status_word || limit_us == 0 || limit_us > 1000000u) return DPARA_ERR_INVALID_ARG;
  dpara::bounded_wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(
      status_word, (uint64_t)limit_us * 1000ull, reinterpret_cast<unsigned long long *>(waited_ns));
  if (cudaGetLastError() != cudaSuccess) return DPARA_ERR_CUDA;
  dpara::count_launches(1);
  return DPARA_OK;
}

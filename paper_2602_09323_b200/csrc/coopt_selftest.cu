// coopt_selftest_bounded_wait: exercises, on its own, the bounded wait that every role of the tcgen05
// kernels uses, so that the time-out path (status word, abort flag, orderly return) can be tested without
// disturbing a real kernel.  One warp waits on an mbarrier that nobody ever arrives on.
#include "coopt_umma.cuh"

namespace coopt {
namespace {

__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(uint64_t limit_ns, int* status, int* elapsed_us) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
    abort_flag = 0;
  }
  __syncwarp();
  const uint64_t t0 = global_timer_ns();
  bool ok = wait_bar(&bar, 0u, &abort_flag, limit_ns);       // phase 0 never completes
  ok = __all_sync(0xffffffffu, ok);
  if (threadIdx.x == 0) {
    if (!ok) atomicCAS(status, 0, COOPT_ERR_TIMEOUT);
    if (elapsed_us) *elapsed_us = static_cast<int>((global_timer_ns() - t0) / 1000ull);
  }
}

}  // namespace
}  // namespace coopt

extern "C" int coopt_selftest_bounded_wait(uint64_t limit_ns, int32_t* status, int32_t* elapsed_us, void* stream) {
  if (!status || limit_ns == 0 || limit_ns > 100000000ull) return COOPT_ERR_INVALID_ARG;   // at most 0.1 s
  coopt::bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(limit_ns, status, elapsed_us);
  return cudaGetLastError() == cudaSuccess ? COOPT_OK : COOPT_ERR_CUDA;
}

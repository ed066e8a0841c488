// Self-test of the bounded device-side wait (not part of the public header).
//
// Every wait inside the tensor-core kernels goes through tc::mbar_wait_for: when its limit runs out the
// waiter records a code in the workspace's status word and returns, and avq_check() reports
// AVQ_ERR_DEVICE_TIMEOUT.  A healthy run never takes that path, so this entry point makes it run once,
// harmlessly: one CTA waits, with a limit of `limit_us` microseconds, on an mbarrier on which nothing will
// ever arrive.  The kernel returns normally after the limit; the context stays usable.
#include "avq_tc_common.cuh"

namespace avq {
namespace {

__global__ void wait_expiry_kernel(int32_t* status_word, unsigned long long limit_ns, int* gave_up) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    tc::mbar_fence_init();
    abort_flag = 0;
  }
  __syncthreads();
  const bool ok = tc::mbar_wait_for(&bar, 0, &abort_flag, status_word, DEV_TIMEOUT_TEST, limit_ns);
  if (!ok && gave_up) atomicAdd(gave_up, 1);
}

}  // namespace
}  // namespace avq

// workspace: a buffer whose first 256 bytes are the status header (an avq_forward workspace works);
// gave_up: optional device int, incremented by every thread whose wait ran out (32 threads wait).
extern "C" __attribute__((visibility("default"))) int32_t avq_selftest_wait_expiry(void* workspace,
                                                                                  uint32_t limit_us,
                                                                                  int* gave_up, void* stream) {
  if (!workspace) return AVQ_ERR_NULL;
  if (limit_us == 0 || limit_us > 100000) return AVQ_ERR_SHAPE;   // at most 0.1 s
  avq::wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<int32_t*>(workspace), (unsigned long long)limit_us * 1000ull, gave_up);
  return cudaGetLastError() == cudaSuccess ? AVQ_OK : AVQ_ERR_CUDA;
}

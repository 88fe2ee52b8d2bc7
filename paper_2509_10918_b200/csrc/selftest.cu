// Test-only entry point: makes a bounded device-side wait run out, the way every wait in the
// tensor-core kernels would if its producer never came, and shows that the kernel then reports
// through the status word and returns instead of hanging.
#include "common.cuh"
#include "tc.cuh"

namespace toma {
namespace {

// One CTA waits, with a limit of `polls` polls, on an mbarrier that nobody arrives at.
__global__ void wait_that_runs_out_kernel(uint32_t polls, uint32_t* dev_status, uint32_t* outcome) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    abort_flag = 0;
    tc::mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool completed = tc::mbar_wait(&bar, 0, dev_status, &abort_flag, polls);
    if (outcome) *outcome = completed ? 1u : 2u;  // 2 = gave up, as it must
  }
}

}  // namespace
}  // namespace toma

extern "C" toma_status toma_test_wait_timeout(uint32_t polls, uint32_t* dev_status, uint32_t* outcome, void* stream) {
  if (polls < 1 || polls > 100000) return TOMA_ERR_SHAPE;
  toma::wait_that_runs_out_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(polls, dev_status, outcome);
  toma::count_launch();
  return cudaGetLastError() == cudaSuccess ? TOMA_OK : TOMA_ERR_CUDA;
}

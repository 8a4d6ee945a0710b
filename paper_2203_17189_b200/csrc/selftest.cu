// Self-test of the bounded waits the tensor-core kernels use.
#include "common.cuh"
#include "tc_common.cuh"

using namespace tc;

// The kernels' bounded wait on a barrier nothing arrives at: the wait gives up after limit_cycles, the CTA records
// code 99 and leaves in the ordinary way.  No loads, no tensor memory: nothing is in flight when it returns.
namespace {
__global__ void selftest_bounded_wait_kernel(int* status, long long limit_cycles) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();
  const bool ok = mbar_wait_limit(&bar, 0, &abort_flag, status, 99, limit_cycles);
  __syncthreads();
  if (ok && threadIdx.x == 0) atomicCAS(status, 0, -1);      // cannot happen: nothing arrives at the barrier
}
}  // namespace

cudaError_t launch_selftest_bounded_wait(int* d_status, long long limit_cycles, cudaStream_t st) {
  selftest_bounded_wait_kernel<<<1, 64, 0, st>>>(d_status, limit_cycles);
  return cudaGetLastError();
}

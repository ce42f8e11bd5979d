// Self-test of the failure path every kernel of the library shares: a bounded wait that runs out,
// the status word it raises, and the early return of whatever is launched while the word is raised.
#include "common.cuh"
#include "ptx.cuh"

namespace pop {
namespace {

// One CTA waits on an mbarrier that nothing ever arrives at, with the same bounded wait the GEMM and
// attention kernels use but a limit given by the caller, records POP_E_DEVICE_TIMEOUT and returns.
__global__ void wait_selftest_kernel(long long limit_cycles, int* __restrict__ status) {
  __shared__ uint64_t bar;
  __shared__ uint32_t raised;
  if (status_raised(status, &raised)) return;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0 && !mbar_wait_limit(&bar, 0, limit_cycles)) atomicMin(status, (int)POP_E_DEVICE_TIMEOUT);
}

}  // namespace
}  // namespace pop

extern "C" int pop_k_wait_selftest(int64_t limit_cycles, void* stream) {
  using namespace pop;
  if (limit_cycles < 1 || limit_cycles > 1000000) return POP_E_INVALID;
  int* status = status_word();
  if (!status) return POP_E_CUDA;
  wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>((long long)limit_cycles, status);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

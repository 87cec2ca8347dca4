// grass_selftest_bounded_wait: exercises the give-up path of the bounded mbarrier wait that
// every pipeline role of the projection kernel uses, without disturbing the GPU: one thread
// waits on a barrier that nothing will ever complete, with a short limit, and records
// GRASS_ERR_TIMEOUT in the status word when the limit runs out.  The kernel returns normally.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace grass {
namespace {

__global__ void bounded_wait_kernel(long long limit_cycles, int* status) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_mbar_init();
    if (!ptx::mbar_wait_bounded(&bar, 0, nullptr, limit_cycles))
      record_status(status, GRASS_ERR_TIMEOUT, 900);
  }
}

}  // namespace
}  // namespace grass

extern "C" int grass_selftest_bounded_wait(int64_t limit_cycles, void* stream) {
  using namespace grass;
  if (limit_cycles < 1 || limit_cycles > 2000000000LL) return GRASS_ERR_INVALID_ARG;
  cudaError_t err;
  int* status = status_word(&err);
  if (status == nullptr) GRASS_CUDA_TRY(err);
  bounded_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(limit_cycles, status);
  GRASS_LAUNCH_CHECK();
  return GRASS_OK;
}

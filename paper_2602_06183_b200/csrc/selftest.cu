// Bounded-wait self-test: the time-out path of the tensor-core kernels, exercised on its own.
// One warp waits with ptx::mbar_wait (the routine every product kernel uses) on an mbarrier that is
// initialised but never completed; when the clock budget is spent the wait returns false, the
// kernel raises the status word exactly as the product kernels do in their teardown, and returns.
#include "sf_common.cuh"
#include "tc_ptx.cuh"

namespace sf {
namespace {

__global__ void __launch_bounds__(32) wait_expiry_kernel(int* status, long long budget) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
  }
  __syncwarp();
  bool ok = true;
  if (threadIdx.x == 0) ok = ptx::mbar_wait(&bar, 0, &abort_flag, budget);   // phase 0 never completes
  __syncwarp();
  if (threadIdx.x == 0 && (!ok || abort_flag)) atomicExch(status, 1);
}

}  // namespace
}  // namespace sf

extern "C" int sf_selftest_wait_expiry(void* workspace, int64_t budget_clocks, void* stream) {
  if (!workspace) return SF_ERR_NULL;
  if (budget_clocks < 1 || budget_clocks > (int64_t(1) << 31)) return SF_ERR_SHAPE;
  if (!sf::aligned16(workspace)) return SF_ERR_ALIGN;
  int st = sf::check_arch();
  if (st != SF_OK) return st;
  sf::wait_expiry_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((int*)workspace, (long long)budget_clocks);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

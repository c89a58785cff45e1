// Self-test of the bounded on-chip wait every tensor-core kernel of the library is built on.
//
// The kernels never block on a hardware barrier: each mbarrier wait polls a limited number of times and,
// when the limit runs out, raises DS_DEV_TIMEOUT in the caller's status word and lets the CTA leave in
// order.  This file exercises exactly that function (mbar_wait_limit) on a barrier nobody arrives on, with
// a small poll limit chosen by the caller, so that the expiry path can be checked without starving a
// barrier inside a real kernel.  One CTA, one warp.
#include "ds_common.cuh"
#include "ds_sm100.cuh"

namespace ds {
namespace {

using namespace sm100;

// report[0] = 1 when the wait on the barrier nobody arrived on gave up, report[1] = polls the abort flag
// then showed (1), report[2] = 1 when, after one arrival, a wait on the same barrier succeeded.
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(uint32_t poll_limit, uint32_t *status, int32_t *report) {
  __shared__ __align__(8) uint64_t bar_storage;
  __shared__ int abort_storage[2];
  const uint32_t bar = smem_u32(&bar_storage);
  volatile int *abort_flag = abort_storage;
  volatile int *abort_flag2 = abort_storage + 1;
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    abort_storage[0] = 0;
    abort_storage[1] = 0;
    fence_barrier_init();
  }
  __syncwarp();
  // phase 0 never completes: every lane's wait has to run out (or see another lane's give-up)
  const bool ok = mbar_wait_limit(bar, 0, abort_flag, poll_limit);
  const bool any_ok = __any_sync(0xffffffffu, ok);
  if (threadIdx.x == 0) {
    if (!any_ok && status != nullptr) atomicOr(status, DS_DEV_TIMEOUT);
    if (report != nullptr) {
      report[0] = any_ok ? 0 : 1;
      report[1] = *abort_flag;
    }
    mbar_arrive(bar);  // now complete the phase: the barrier is still usable after the expired wait
  }
  __syncwarp();
  const bool ok2 = mbar_wait_limit(bar, 0, abort_flag2, kSpinLimit);
  const bool all_ok2 = __all_sync(0xffffffffu, ok2);
  if (threadIdx.x == 0 && report != nullptr) report[2] = all_ok2 ? 1 : 0;
}

}  // namespace

int launch_bounded_wait_selftest(uint32_t poll_limit, uint32_t *status, int32_t *report, cudaStream_t stream) {
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(poll_limit, status, report);
  DS_CUDA_OK(cudaGetLastError());
  note_launch(1);
  return DS_OK;
}

}  // namespace ds

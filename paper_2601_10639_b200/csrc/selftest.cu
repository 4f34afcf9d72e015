// Self-test of the bounded wait every pipeline role of the contraction kernels relies on: one
// thread waits on an mbarrier that nobody completes, gives up after the limit and records
// STEM_ERR_TIMEOUT in the status word, exactly as a stalled pipeline role would.  Nothing is
// in flight (no TMA copy, no MMA, no other CTA), so giving up needs no unwinding and the
// context stays usable.  With `arrive` set the barrier is completed first and the wait must
// succeed: the same code path, the other outcome.
#include "ptx_sm100.cuh"
#include "stem_internal.h"

namespace stem {
namespace {

__global__ void __launch_bounds__(32)
selftest_wait_kernel(int32_t* status, long long limit_cycles, int arrive) {
  __shared__ __align__(8) uint64_t bar_storage;
  __shared__ int abort_flag;
  const uint32_t bar = ptx::smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    ptx::mbar_init(bar, 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (arrive) ptx::mbar_arrive(bar);      // phase 0 completes: the wait below returns at once
    if (!ptx::mbar_wait_bounded(bar, 0u, &abort_flag, limit_cycles)) report_error(status, STEM_ERR_TIMEOUT, 100);
  }
}

}  // namespace

cudaError_t launch_selftest_wait(int32_t* status, long long limit_cycles, int arrive, cudaStream_t stream) {
  selftest_wait_kernel<<<1, 32, 0, stream>>>(status, limit_cycles, arrive);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace stem

// Test aids that need a kernel of their own.
//
// qgalore_debug_expire_wait: every tensor-core kernel of the library waits on its shared-memory barriers
// with a poll limit and, when a wait runs out, raises QG_DEV_WAIT_EXPIRED in the caller's status word and
// winds down.  That path cannot be provoked in the real kernels without abandoning copies in flight, so it
// is exercised here in its harmless form: one warp, one barrier that nothing ever signals, no asynchronous
// copy outstanding, no tensor memory held.  The wait is the same try_wait loop, with the limit as an argument.
#include "qg_common.cuh"
#include "sm100_ptx.cuh"

namespace qg {
namespace {

__global__ void __launch_bounds__(32)
expire_wait_kernel(uint32_t polls, int32_t* __restrict__ status, int32_t* __restrict__ polls_used) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_mbar_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    uint32_t i = 0;
    bool done = false;
    for (; i < polls && !done; ++i) done = ptx::mbar_try_wait(&bar, 0);   // phase 0 never completes: nobody arrives
    if (polls_used) *polls_used = (int32_t)i;
    if (!done && status) atomicOr(status, QG_DEV_WAIT_EXPIRED);
  }
}

}  // namespace
}  // namespace qg

extern "C" int qgalore_debug_expire_wait(int32_t polls, int32_t* status_dev, int32_t* polls_used_dev, void* stream) {
  using namespace qg;
  if (polls < 1 || polls > (1 << 20) || !status_dev) return QG_INVALID_ARGUMENT;
  if (!aligned4(status_dev) || (polls_used_dev && !aligned4(polls_used_dev))) return QG_MISALIGNED;
  expire_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((uint32_t)polls, status_dev, polls_used_dev);
  QG_LAUNCH_CHECK();
  return QG_OK;
}

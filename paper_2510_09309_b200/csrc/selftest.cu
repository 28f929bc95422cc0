// Self-test of the bounded waits: one thread waits on an mbarrier that nothing ever arrives at.  The wait must give up
// after its limit (about one second), raise MASKKV_FLAG_TIMEOUT, record where it gave up and let the kernel return -
// a lost signal ends in a status word the host can read, never in a hang, and the context stays usable.
#include "selftest.h"

#include "tc_common.cuh"

namespace mkv {
namespace tc {

namespace {
__global__ void wait_expiry_kernel(uint32_t* __restrict__ status) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_word;
  volatile uint32_t* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    *abort_flag = 0u;
    fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) (void)mbar_wait(&bar, 0, abort_flag, status, kSelftestWhere);
  __syncthreads();
}
}  // namespace

void launch_wait_expiry_selftest(maskkv_ctx* ctx, cudaStream_t st) {
  wait_expiry_kernel<<<1, 32, 0, st>>>(ctx->status_dev);
}

}  // namespace tc
}  // namespace mkv

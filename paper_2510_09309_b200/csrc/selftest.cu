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
// Measures the rate of the special-function unit: every thread runs eight independent chains of ex2.approx.ftz.f32
// (the instruction both scoring sweeps spend their time on), `iters` rounds of them; the sums keep the chains alive.
__global__ void __launch_bounds__(1024, 1) ex2_rate_kernel(float* __restrict__ out, int iters) {
  float x[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) x[u] = -1.0f - 0.001f * (float)(threadIdx.x + u);
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
#pragma unroll
      for (int u = 0; u < 8; ++u) x[u] = ex2(x[u]) - 1.5f;   // stays in [-1.5, -0.5]
    }
  }
  float acc = 0.f;
#pragma unroll
  for (int u = 0; u < 8; ++u) acc += x[u];
  if (acc == 12345.678f) out[0] = acc;                     // never true: the result only has to be observable
}
}  // namespace

long long launch_ex2_rate_selftest(maskkv_ctx* ctx, float* out, int iters, cudaStream_t st) {
  const int grid = ctx->sm_count * 2;
  ex2_rate_kernel<<<grid, 1024, 0, st>>>(out, iters);
  return (long long)grid * 1024 * 32 * iters;              // exponentials evaluated
}

void launch_wait_expiry_selftest(maskkv_ctx* ctx, cudaStream_t st) {
  wait_expiry_kernel<<<1, 32, 0, st>>>(ctx->status_dev);
}

}  // namespace tc
}  // namespace mkv

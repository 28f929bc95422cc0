// Host-side entry point of the bounded-wait self-test (selftest.cu), used by maskkv_api.cu.
#pragma once

#include "common.cuh"

namespace mkv {
namespace tc {

constexpr uint32_t kSelftestWhere = 0x7e57u;   // the "where" code the expired wait records in status word 1

void launch_wait_expiry_selftest(maskkv_ctx* ctx, cudaStream_t st);
// Enqueues the exponential-rate measurement; returns how many exponentials the launch evaluates.
long long launch_ex2_rate_selftest(maskkv_ctx* ctx, float* out, int iters, cudaStream_t st);

}  // namespace tc
}  // namespace mkv

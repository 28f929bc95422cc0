// Host-side entry point of the bounded-wait self-test (selftest.cu), used by maskkv_api.cu.
#pragma once

#include "common.cuh"

namespace mkv {
namespace tc {

constexpr uint32_t kSelftestWhere = 0x7e57u;   // the "where" code the expired wait records in status word 1

void launch_wait_expiry_selftest(maskkv_ctx* ctx, cudaStream_t st);

}  // namespace tc
}  // namespace mkv

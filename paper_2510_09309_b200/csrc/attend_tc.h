// Host-side entry points of the tensor-core attention kernel (attend_tc.cu), used by maskkv_api.cu.
#pragma once

#include "common.cuh"

namespace mkv {
namespace tc {

bool attend_tc_supported(const maskkv_ctx* ctx, const Shape& sh);
// Returns 0 after a launch, 1 when nothing was launched (tensor map or attribute set-up failed).
// cache_rows = rows allocated in kc / vc (reads never go past them).  q_cu (device) = cumulative query rows per
// request, sum_q / max_q their total and largest count: the live rows (q_cu = live_cu) or a subset of them.
int launch_attend_tc(maskkv_ctx* ctx, const Shape& sh, const void* q, const int32_t* q_cu, int sum_q, int max_q, const void* kl,
                     const void* vl, const void* kc, const void* vc, long long cache_rows, const int32_t* offsets, void* out,
                     float* lse, cudaStream_t st);

}  // namespace tc
}  // namespace mkv

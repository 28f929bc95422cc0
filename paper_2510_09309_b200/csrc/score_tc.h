// Host-side entry points of the tensor-core scoring kernels (score_tc.cu), used by maskkv_api.cu.
#pragma once

#include "common.cuh"

namespace mkv {
namespace tc {

// True when the tcgen05 path can serve this problem (bf16, tensor-map encoder resolved, voters present).
bool score_tc_supported(const maskkv_ctx* ctx, const Shape& sh);
// Upper bounds used to size the workspace: partials per row in sweep 1, key tiles per request in sweep 2.
int score_tc_max_chunks(const maskkv_ctx* ctx, const Shape& sh);
int score_tc_max_tiles(const Shape& sh);

// Each returns 0 after its launches, 1 when nothing was launched (tensor map or attribute set-up failed).
// The *_host arrays are the descriptor's cumulative lengths.
// Sweep 1 leaves per-CTA partials in `part` and clears the R*H_kv words of `seg_cnt` that sweep 2 counts in.
int launch_score_stats_tc(maskkv_ctx* ctx, const Shape& sh, const int32_t* prompt_cu_host, const int32_t* live_cu_host,
                          const void* q, const void* kp, const void* km, float2* part, int C, uint32_t* seg_cnt, cudaStream_t st);
// part -> lse, for a sweep 2 that is not the tensor-core kernel.
void launch_score_merge_tc(maskkv_ctx* ctx, const Shape& sh, const int32_t* prompt_cu_host, const int32_t* live_cu_host,
                           const float2* part, int C, float* lse, cudaStream_t st);
// Sweep 2.  Row normalisers come from `part` (sweep 1's partials, merged in the kernel) when it is not null, else from
// `lse`.  With one query block per KV head (no grouped heads, at most 256 voters per request) it writes scores and -
// the warp that finishes a segment's last tile adds up its partials - mass_p / mass_m; `seg_cnt` (R*H_kv words) must
// be zero on entry.  With several blocks (score_tc_split_blocks) each block's column sums go to `colpart`
// (score_tc_colpart_bytes), a second kernel adds them into scores and leaves per-tile mass partials in `mass_part` in
// the layout score_mass_reduce reads: the caller launches that kernel afterwards.  scores_live (may be null) receives the
// column sums over the live keys, [H_kv][sum_M].  *launches = kernels launched.
bool score_tc_split_blocks(const Shape& sh);
size_t score_tc_colpart_bytes(const Shape& sh);
int launch_score_colsum_tc(maskkv_ctx* ctx, const Shape& sh, const int32_t* prompt_cu_host, const int32_t* live_cu_host,
                           const void* q, const void* kp, const void* km, const float* lse, const float2* part, int C,
                           const float* w, float* scores, float* colpart, float2* mass_part, int Tmax, uint32_t* seg_cnt,
                           float* mass_p, float* mass_m, float* scores_live, bool any_without_voters, cudaStream_t st, int* launches);

}  // namespace tc
}  // namespace mkv

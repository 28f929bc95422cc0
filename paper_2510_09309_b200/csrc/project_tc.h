// Host-side entry points of the mask-only projection (project_tc.cu), used by maskkv_api.cu.
#pragma once

#include "common.cuh"

namespace mkv {
namespace tc {

// True when the context can run the tensor-core GEMM (tensor-map encoder resolved, enough shared memory).
bool project_tc_supported(const maskkv_ctx* ctx);
// Gather (when positions != nullptr; `packed` then holds n_mask * width bf16) + GEMM.  Strides in elements.
// Returns 0 after its launches, 1 when nothing was launched (tensor map or attribute set-up failed).
int launch_project_tc(maskkv_ctx* ctx, const void* hidden, long long n_tokens, int width, long long hidden_row_stride,
                      const int32_t* positions, int n_mask, const void* w_vocab, int vocab, long long w_row_stride, void* out,
                      long long ld_out, int out_bf16, void* packed, cudaStream_t st, int* launches);

// The GEMM on pairs of CTAs (project_tc2.cu): a_base = the packed rows (or the hidden rows in place), byte stride.
// Returns 0 after its launch, 1 when nothing was launched.
bool project_tc2_supported(const maskkv_ctx* ctx);
int launch_project_gemm_tc2(maskkv_ctx* ctx, const void* a_base, long long a_stride_bytes, int width, int n_mask, const void* w_vocab,
                            int vocab, long long w_row_stride, void* out, long long ld_out, int out_bf16, cudaStream_t st);

}  // namespace tc
}  // namespace mkv

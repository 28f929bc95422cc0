// Layer importance (Eq. 8): I = 1 - mean_i cos(h_in_i, h_out_i) over the token rows of one layer - the offline
// profile that maskkv_layer_budgets consumes.  A streaming reduction bound by HBM: every element of the two
// hidden-state tensors is read exactly once, 16 bytes per lane per access, eight accesses per tensor in flight.
//
// One warp per token row (grid-stride); a warp adds the cosines of its rows in row order into a double, the block
// adds its warps in warp order, and a second one-block kernel adds the block partials in a fixed tree: the result
// does not depend on scheduling.  A row with a zero vector counts as cosine 0.
#pragma once

#include "common.cuh"

namespace mkv {

constexpr int kImpThreads = 256;
constexpr int kImpBlocksPerSm = 4;

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

template <typename T> struct ImpVec;
template <> struct ImpVec<float> {
  static constexpr int kElems = 4;
  __device__ static __forceinline__ void acc(const uint4& a, const uint4& b, float& dot, float& na, float& nb) {
    const float x[4] = {__uint_as_float(a.x), __uint_as_float(a.y), __uint_as_float(a.z), __uint_as_float(a.w)};
    const float y[4] = {__uint_as_float(b.x), __uint_as_float(b.y), __uint_as_float(b.z), __uint_as_float(b.w)};
#pragma unroll
    for (int t = 0; t < 4; ++t) { dot = fmaf(x[t], y[t], dot); na = fmaf(x[t], x[t], na); nb = fmaf(y[t], y[t], nb); }
  }
};
template <> struct ImpVec<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ static __forceinline__ void acc(const uint4& a, const uint4& b, float& dot, float& na, float& nb) {
    const uint32_t wa[4] = {a.x, a.y, a.z, a.w}, wb[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float x0 = __uint_as_float(wa[t] << 16), x1 = __uint_as_float(wa[t] & 0xffff0000u);
      const float y0 = __uint_as_float(wb[t] << 16), y1 = __uint_as_float(wb[t] & 0xffff0000u);
      dot = fmaf(x0, y0, dot); dot = fmaf(x1, y1, dot);
      na = fmaf(x0, x0, na); na = fmaf(x1, x1, na);
      nb = fmaf(y0, y0, nb); nb = fmaf(y1, y1, nb);
    }
  }
};

// partial[block] = sum of cos over the rows this block's warps visited
template <typename T>
__global__ void __launch_bounds__(kImpThreads)
importance_partial_kernel(const T* __restrict__ h_in, const T* __restrict__ h_out, long long n_tokens, int hidden,
                          long long in_stride, long long out_stride, double* __restrict__ partial) {
  __shared__ double warp_sum_s[kImpThreads / 32];
  constexpr int E = ImpVec<T>::kElems;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int vecs = hidden / E;                            // 16-byte pieces per row
  const long long warps_total = (long long)gridDim.x * (kImpThreads / 32);
  double cos_sum = 0.0;
  for (long long row = (long long)blockIdx.x * (kImpThreads / 32) + warp; row < n_tokens; row += warps_total) {
    const uint4* a = reinterpret_cast<const uint4*>(h_in + row * in_stride);
    const uint4* b = reinterpret_cast<const uint4*>(h_out + row * out_stride);
    float dot = 0.f, na = 0.f, nb = 0.f;
    for (int v0 = lane; v0 < vecs; v0 += 32 * 8) {
      uint4 va[8], vb[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int v = v0 + u * 32;
        if (v < vecs) { va[u] = ld_stream16(a + v); vb[u] = ld_stream16(b + v); }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int v = v0 + u * 32;
        if (v < vecs) ImpVec<T>::acc(va[u], vb[u], dot, na, nb);
      }
    }
    dot = warp_sum(dot); na = warp_sum(na); nb = warp_sum(nb);
    const float den = sqrtf(na) * sqrtf(nb);
    cos_sum += den > 0.f ? (double)(dot / den) : 0.0;
  }
  if (lane == 0) warp_sum_s[warp] = cos_sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < kImpThreads / 32; ++w) s += warp_sum_s[w];
    partial[blockIdx.x] = s;
  }
}

// One block: thread t adds partial[t], partial[t + 256], ... in that order, the warp adds its lanes through a fixed
// shuffle tree, thread 0 adds the warps in warp order.
__global__ void __launch_bounds__(kImpThreads)
importance_final_kernel(const double* __restrict__ partial, int n_blocks, long long n_tokens, float* __restrict__ out) {
  __shared__ double warp_sum_s[kImpThreads / 32];
  double s = 0.0;
  for (int b = threadIdx.x; b < n_blocks; b += kImpThreads) s += partial[b];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) warp_sum_s[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < kImpThreads / 32; ++w) t += warp_sum_s[w];
    *out = n_tokens > 0 ? (float)(1.0 - t / (double)n_tokens) : 0.f;
  }
}

}  // namespace mkv

// Response-token refresh rule of the feature cache the method builds on (appendix, "Response tokens"):
//     S_shift = { i : cos(V_i^(t), V_i^(t-1)) < delta },   S = S_shift, or every row on a periodic-refresh step.
// Two small kernels: a warp per token row forms the cosine (same streaming loads and accumulation as the layer
// importance kernel) and leaves a 0/1 flag in idx[i]; one block then turns the flags into the ascending index list
// in place, 4096 rows per round (every flag of a round is read before any index of that round is written, and an
// index never lands behind its own row, so unread flags are never overwritten).
#pragma once

#include "importance.cuh"

namespace mkv {

constexpr int kRefreshThreads = 256;
constexpr int kRefreshScanThreads = 1024;
constexpr int kRefreshItems = 4;                        // rows per thread and round of the compaction

template <typename T>
__global__ void __launch_bounds__(kRefreshThreads)
refresh_flag_kernel(const T* __restrict__ v_cur, const T* __restrict__ v_prev, long long n_tokens, int width,
                    long long cur_stride, long long prev_stride, float delta, int refresh_all,
                    float* __restrict__ cos_out, int32_t* __restrict__ idx) {
  constexpr int E = ImpVec<T>::kElems;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int vecs = width / E;
  const long long warps_total = (long long)gridDim.x * (kRefreshThreads / 32);
  pdl_launch_dependents();                                 // the compaction kernel may set itself up meanwhile
  for (long long row = (long long)blockIdx.x * (kRefreshThreads / 32) + warp; row < n_tokens; row += warps_total) {
    float cosv = 0.f;
    if (!refresh_all || cos_out != nullptr) {
      const uint4* a = reinterpret_cast<const uint4*>(v_cur + row * cur_stride);
      const uint4* b = reinterpret_cast<const uint4*>(v_prev + row * prev_stride);
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
      cosv = den > 0.f ? dot / den : 0.f;                   // a zero row counts as cosine 0
    }
    if (lane == 0) {
      if (cos_out != nullptr) cos_out[row] = cosv;
      idx[row] = (refresh_all || cosv < delta) ? 1 : 0;
    }
  }
}

// One block.  idx[0..n) holds flags on entry, the ascending indices of the flagged rows in idx[0..count) on exit.
// A thread owns kRefreshItems consecutive rows of a round.
__global__ void __launch_bounds__(kRefreshScanThreads)
refresh_compact_kernel(long long n_tokens, int32_t* __restrict__ idx, int32_t* __restrict__ count) {
  __shared__ int warp_tot[kRefreshScanThreads / 32];
  __shared__ int base_s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) base_s = 0;
  pdl_wait();                                              // the flags come from the previous kernel of the stream
  __syncthreads();
  for (long long r0 = 0; r0 < n_tokens; r0 += kRefreshScanThreads * kRefreshItems) {
    const long long row0 = r0 + (long long)tid * kRefreshItems;
    int flags = 0;                                         // bit k: row0 + k is flagged
#pragma unroll
    for (int k = 0; k < kRefreshItems; ++k)
      if (row0 + k < n_tokens && idx[row0 + k] != 0) flags |= 1 << k;
    const int mine = __popc(flags);
    int incl = mine;                                       // inclusive prefix over the warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();                                       // every flag of the round has been read
    int pos = base_s + incl - mine;
    for (int w = 0; w < warp; ++w) pos += warp_tot[w];
#pragma unroll
    for (int k = 0; k < kRefreshItems; ++k)
      if ((flags >> k) & 1) idx[pos++] = (int32_t)(row0 + k);
    __syncthreads();
    if (tid == 0) {
      int t = base_s;
      for (int w = 0; w < kRefreshScanThreads / 32; ++w) t += warp_tot[w];
      base_s = t;
    }
    __syncthreads();
  }
  if (tid == 0) *count = base_s;
}

}  // namespace mkv

// Attention of a later denoising step over [compacted prompt segment ; live keys] on the plain FP32
// pipes: the fp32 path, and the formulation the tensor-core path is checked against.
//
// One warp per query row; the lanes split head_dim.  Keys are visited four at a time with an online
// (running max / running sum) softmax, so the weights never leave registers.
#pragma once

#include "common.cuh"

namespace mkv {

constexpr int kAttendWarps = 8;

template <typename T, int E>
__device__ __forceinline__ void load_lane(const T* p, float* dst);
template <>
__device__ __forceinline__ void load_lane<float, 2>(const float* p, float* dst) {
  const float2 v = *reinterpret_cast<const float2*>(p); dst[0] = v.x; dst[1] = v.y;
}
template <>
__device__ __forceinline__ void load_lane<float, 4>(const float* p, float* dst) {
  const float4 v = *reinterpret_cast<const float4*>(p); dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
}
template <>
__device__ __forceinline__ void load_lane<__nv_bfloat16, 2>(const __nv_bfloat16* p, float* dst) {
  const uint32_t w = *reinterpret_cast<const uint32_t*>(p);
  dst[0] = __uint_as_float(w << 16); dst[1] = __uint_as_float(w & 0xffff0000u);
}
template <>
__device__ __forceinline__ void load_lane<__nv_bfloat16, 4>(const __nv_bfloat16* p, float* dst) {
  const uint2 w = *reinterpret_cast<const uint2*>(p);
  dst[0] = __uint_as_float(w.x << 16); dst[1] = __uint_as_float(w.x & 0xffff0000u);
  dst[2] = __uint_as_float(w.y << 16); dst[3] = __uint_as_float(w.y & 0xffff0000u);
}

// grid (ceil(largest query count / kAttendWarps), H, R); block kAttendWarps * 32.
template <typename T, int D>
__global__ void __launch_bounds__(kAttendWarps * 32)
attend_simt(Shape sh, const T* __restrict__ q, const T* __restrict__ kl, const T* __restrict__ vl,
            const T* __restrict__ kc, const T* __restrict__ vc, const int32_t* __restrict__ offsets,
            const int32_t* __restrict__ q_cu, int sum_q, long long capacity, T* __restrict__ out, float* __restrict__ lse,
            uint32_t* __restrict__ status) {
  constexpr int E = D / 32;
  const int lane = threadIdx.x & 31;
  const int h = blockIdx.y, r = blockIdx.z, hk = h / sh.g;
  const int l0 = sh.live_cu[r], M = sh.live_cu[r + 1] - l0;
  const int ql0 = q_cu[r], Mq = q_cu[r + 1] - ql0;          // the query rows: the live rows or a subset of them
  const int i = blockIdx.x * kAttendWarps + (threadIdx.x >> 5);
  if (i >= Mq) return;
  const int s = r * sh.Hkv + hk;
  // rows [c0, c0 + nc) of the cache; offsets that point outside the `capacity` rows the cache holds are clipped and
  // flagged, never dereferenced
  long long c0 = offsets[s], c1 = offsets[s + 1];
  if (c0 < 0 || c1 < c0 || c1 > capacity) {
    if (lane == 0) atomicOr(status, (uint32_t)MASKKV_FLAG_BOUNDS);
    c0 = c0 < 0 ? 0 : (c0 > capacity ? capacity : c0);
    c1 = c1 < c0 ? c0 : (c1 > capacity ? capacity : c1);
  }
  const int nc = (int)(c1 - c0);
  const int total = nc + M;

  float qv[E], acc[E];
  load_lane<T, E>(q + (long long)(ql0 + i) * sh.q_ts + (long long)h * sh.q_hs + lane * E, qv);
#pragma unroll
  for (int e = 0; e < E; ++e) { qv[e] *= sh.scale; acc[e] = 0.f; }
  float m = -INFINITY, l = 0.f;

  auto krow = [&](int j) -> const T* {
    return j < nc ? kc + (long long)(c0 + j) * D + lane * E
                  : kl + (long long)(l0 + j - nc) * sh.kv_ts + (long long)hk * sh.kv_hs + lane * E;
  };
  auto vrow = [&](int j) -> const T* {
    return j < nc ? vc + (long long)(c0 + j) * D + lane * E
                  : vl + (long long)(l0 + j - nc) * sh.kv_ts + (long long)hk * sh.kv_hs + lane * E;
  };

  for (int j0 = 0; j0 < total; j0 += 4) {
    float sc[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float part = 0.f;
      if (j0 + u < total) {
        float kv[E];
        load_lane<T, E>(krow(j0 + u), kv);
#pragma unroll
        for (int e = 0; e < E; ++e) part = fmaf(qv[e], kv[e], part);
      }
      sc[u] = part;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
      for (int u = 0; u < 4; ++u) sc[u] += __shfl_xor_sync(0xffffffffu, sc[u], o);
    }
    float m_new = m;
#pragma unroll
    for (int u = 0; u < 4; ++u) if (j0 + u < total) m_new = fmaxf(m_new, sc[u]);
    const float corr = expf(m - m_new);                  // m = -inf at the start gives 0
    l *= corr;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] *= corr;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (j0 + u < total) {
        const float p = expf(sc[u] - m_new);
        float vv[E];
        load_lane<T, E>(vrow(j0 + u), vv);
        l += p;
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = fmaf(p, vv[e], acc[e]);
      }
    }
    m = m_new;
  }
  const float inv = 1.f / l;
  T* o = out + (long long)(ql0 + i) * sh.q_ts + (long long)h * sh.q_hs + lane * E;
#pragma unroll
  for (int e = 0; e < E; ++e) o[e] = from_f32<T>(acc[e] * inv);
  if (lse != nullptr && lane == 0) lse[(long long)h * sum_q + ql0 + i] = m + logf(l);
}

}  // namespace mkv

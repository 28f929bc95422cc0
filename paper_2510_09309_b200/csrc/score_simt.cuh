// Mask-voting scores (Eq. 6-7, sums of Eq. 14) on the plain FP32 pipes.
// This is the fp32 path (tensor cores have no fp32 product that holds 1e-5) and the reference
// formulation the tensor-core path is checked against on the device.
//
// Two sweeps over the logits, neither of which stores them:
//   1. score_stats_simt   : thread = one mask query (row held in registers), keys streamed through
//                           shared memory; per key chunk a partial (row max, sum of exp).
//      score_merge_stats  : log-sum-exp merge of the chunk partials -> lse_i = m_i + ln l_i.
//   2. score_colsum_simt  : thread = one key (row in registers), queries streamed through shared
//                           memory; A_ij = exp(s_ij - lse_i) is summed over i in the owning thread,
//                           so the column sum needs no cross-thread reduction.
//      score_mass_reduce  : fixed-order reduction of the per-block mass partials (deterministic).
#pragma once

#include "common.cuh"

namespace mkv {

constexpr int kSimtThreads = 128;
constexpr int kSimtStage = 32;      // rows staged in shared memory per step
constexpr int kStatsChunk = 512;    // keys per partial in sweep 1

template <typename T, int D>
__device__ __forceinline__ const T* key_row(const Shape& sh, const T* kp, const T* km, int p0, int l0, int N,
                                            int hk, int j) {
  return j < N ? kp + (long long)(p0 + j) * sh.kv_ts + (long long)hk * sh.kv_hs
               : km + (long long)(l0 + j - N) * sh.kv_ts + (long long)hk * sh.kv_hs;
}

template <int D>
__device__ __forceinline__ float dot_smem(const float* reg, const float* __restrict__ row) {
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
  for (int c = 0; c < D; c += 4) {
    float4 v = *reinterpret_cast<const float4*>(row + c);
    a0 = fmaf(reg[c], v.x, a0);
    a1 = fmaf(reg[c + 1], v.y, a1);
    a2 = fmaf(reg[c + 2], v.z, a2);
    a3 = fmaf(reg[c + 3], v.w, a3);
  }
  return (a0 + a1) + (a2 + a3);
}

// grid (chunks, H, R * q_tiles); block kSimtThreads.  part[(h*sumM + row)*C + chunk] = (max, sum).
template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
score_stats_simt(Shape sh, const T* __restrict__ q, const T* __restrict__ kp, const T* __restrict__ km,
                 float2* __restrict__ part, int C) {
  __shared__ __align__(16) float ks[kSimtStage][D];
  const int q_tiles = (sh.maxM + kSimtThreads - 1) / kSimtThreads;
  const int c = blockIdx.x, h = blockIdx.y, r = blockIdx.z / q_tiles, qt = blockIdx.z % q_tiles;
  const int hk = h / sh.g;
  const int p0 = sh.prompt_cu[r], N = sh.prompt_cu[r + 1] - p0;
  const int l0 = sh.live_cu[r], M = sh.live_cu[r + 1] - l0;
  const int i = qt * kSimtThreads + threadIdx.x;
  const bool valid = i < M;
  if (qt * kSimtThreads >= M) return;                 // whole block idle (uniform)
  const int k0 = c * kStatsChunk;
  const int k1 = min(k0 + kStatsChunk, N + M);

  float qreg[D];
  if (valid) load_row<D>(q + (long long)(l0 + i) * sh.q_ts + (long long)h * sh.q_hs, qreg);
  else {
#pragma unroll
    for (int t = 0; t < D; ++t) qreg[t] = 0.f;
  }
  float m = -INFINITY, l = 0.f;
  for (int kt = k0; kt < k1; kt += kSimtStage) {
    const int rows = min(kSimtStage, k1 - kt);
    // stage `rows` key rows as fp32: D/4 float4 slots per row
    for (int e = threadIdx.x; e < rows * (D / 8); e += kSimtThreads) {
      const int jr = e / (D / 8), cc = (e % (D / 8)) * 8;
      float tmp[8];
      load_row<8>(key_row<T, D>(sh, kp, km, p0, l0, N, hk, kt + jr) + cc, tmp);
#pragma unroll
      for (int t = 0; t < 8; ++t) ks[jr][cc + t] = tmp[t];
    }
    __syncthreads();
    for (int jr = 0; jr < rows; ++jr) {
      const float s = dot_smem<D>(qreg, ks[jr]) * sh.scale;
      if (s > m) { l = l * expf(m - s) + 1.f; m = s; }
      else l += expf(s - m);
    }
    __syncthreads();
  }
  if (valid) part[((long long)h * sh.sumM + l0 + i) * C + c] = make_float2(m, l);
}

// One thread per (h, row): lse[h*sumM + row] = ln sum_j exp(s_j), from partials that cover kStatsChunk keys each.
__global__ void score_merge_stats(Shape sh, const float2* __restrict__ part, int C, float* __restrict__ lse) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= (long long)sh.H * sh.sumM) return;
  const int row = (int)(t % sh.sumM);
  const int r = find_request(sh.live_cu, sh.R, row);
  const int N = sh.prompt_cu[r + 1] - sh.prompt_cu[r], M = sh.live_cu[r + 1] - sh.live_cu[r];
  const int chunks = (N + M + kStatsChunk - 1) / kStatsChunk;
  const float2* p = part + t * C;
  float m = -INFINITY;
  for (int c = 0; c < chunks; ++c) m = fmaxf(m, p[c].x);
  float l = 0.f;
  for (int c = 0; c < chunks; ++c) l += p[c].y * expf(p[c].x - m);
  lse[t] = m + logf(l);
}

// grid (key tiles, H_kv, R); block kSimtThreads.  mass_part[(s*Tmax + tile)*4 + slot] = (prompt sum, mask sum),
// s = r*H_kv + hk; this kernel puts the tile's total in slot 0 (the tensor-core kernel fills one slot per warp).
template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
score_colsum_simt(Shape sh, const T* __restrict__ q, const T* __restrict__ kp, const T* __restrict__ km,
                  const float* __restrict__ lse, const float* __restrict__ w, float* __restrict__ scores,
                  float* __restrict__ scores_live, float2* __restrict__ mass_part, int Tmax) {
  __shared__ __align__(16) float qs[kSimtStage][D];
  __shared__ float ls[kSimtStage], ws[kSimtStage];
  __shared__ float red[2][kSimtThreads / 32];
  const int tile = blockIdx.x, hk = blockIdx.y, r = blockIdx.z;
  const int p0 = sh.prompt_cu[r], N = sh.prompt_cu[r + 1] - p0;
  const int l0 = sh.live_cu[r], M = sh.live_cu[r + 1] - l0;
  float2* mp = mass_part + ((long long)(r * sh.Hkv + hk) * Tmax + tile) * 4;
  if (threadIdx.x < 4) mp[threadIdx.x] = make_float2(0.f, 0.f);
  if (tile * kSimtThreads >= N + M) return;            // beyond this request's keys (uniform)
  const int j = tile * kSimtThreads + threadIdx.x;
  const bool valid = j < N + M;
  float kreg[D];
  if (valid) load_row<D>(key_row<T, D>(sh, kp, km, p0, l0, N, hk, j), kreg);
  else {
#pragma unroll
    for (int t = 0; t < D; ++t) kreg[t] = 0.f;
  }
  float acc = 0.f;
  for (int h = hk * sh.g; h < (hk + 1) * sh.g; ++h) {
    for (int i0 = 0; i0 < M; i0 += kSimtStage) {
      const int rows = min(kSimtStage, M - i0);
      for (int e = threadIdx.x; e < rows * (D / 8); e += kSimtThreads) {
        const int ir = e / (D / 8), cc = (e % (D / 8)) * 8;
        float tmp[8];
        load_row<8>(q + (long long)(l0 + i0 + ir) * sh.q_ts + (long long)h * sh.q_hs + cc, tmp);
#pragma unroll
        for (int t = 0; t < 8; ++t) qs[ir][cc + t] = tmp[t];
      }
      if (threadIdx.x < rows) {
        ls[threadIdx.x] = lse[(long long)h * sh.sumM + l0 + i0 + threadIdx.x];
        ws[threadIdx.x] = w ? w[l0 + i0 + threadIdx.x] : 1.f;
      }
      __syncthreads();
      for (int ir = 0; ir < rows; ++ir) {
        const float s = dot_smem<D>(kreg, qs[ir]) * sh.scale;
        acc = fmaf(ws[ir], expf(s - ls[ir]), acc);
      }
      __syncthreads();
    }
  }
  if (valid && j < N) scores[(long long)hk * sh.sumN + p0 + j] = acc;
  if (valid && j >= N && scores_live != nullptr) scores_live[(long long)hk * sh.sumM + l0 + (j - N)] = acc;
  float sp = (valid && j < N) ? acc : 0.f;
  float sm = (valid && j >= N) ? acc : 0.f;
  sp = warp_sum(sp);
  sm = warp_sum(sm);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = sp; red[1][threadIdx.x >> 5] = sm; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.f, b = 0.f;
    for (int t = 0; t < kSimtThreads / 32; ++t) { a += red[0][t]; b += red[1][t]; }
    *mp = make_float2(a, b);
  }
}

// One warp per segment s: fixed-order sum of the tile partials (4 slots per tile) of the request's own tiles.
__global__ void score_mass_reduce(Shape sh, const float2* __restrict__ mass_part, int Tmax,
                                  float* __restrict__ mass_p, float* __restrict__ mass_m) {
  const int s = blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5);
  if (s >= sh.R * sh.Hkv) return;
  const int lane = threadIdx.x & 31;
  const int r = s / sh.Hkv;
  const int N = sh.prompt_cu[r + 1] - sh.prompt_cu[r], M = sh.live_cu[r + 1] - sh.live_cu[r];
  const int entries = ((N + 127) / 128 + (M + 127) / 128) * 4;
  float a = 0.f, b = 0.f;
  for (int t = lane; t < entries; t += 32) {
    const float2 v = mass_part[(long long)s * Tmax * 4 + t];
    a += v.x;
    b += v.y;
  }
  a = warp_sum(a);
  b = warp_sum(b);
  if (lane == 0) { mass_p[s] = a; mass_m[s] = b; }
}

}  // namespace mkv

// Top-k eviction (Eq. 16): an exact radix select per (request, head) segment.
//
// One block per segment.  The segment's scores are turned into order-preserving 32-bit keys and
// (when they fit) staged once in shared memory; four 8-bit histogram passes then find the k-th
// largest key exactly, and a last sweep emits the kept indices in ascending order, ties at the
// threshold going to the lowest indices.  Each warp owns a contiguous index range and walks it 32
// consecutive elements at a time, so ranks inside a step come from a ballot and shared-memory
// accesses are conflict-free.
#pragma once

#include "common.cuh"

namespace mkv {

constexpr int kSelectThreads = 1024;
constexpr int kSelectWarps = kSelectThreads / 32;

// Larger float <=> larger key; NaN maps to 0 (below every number, -inf included).
__device__ __forceinline__ uint32_t order_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;
  if (u == 0x80000000u) u = 0u;                          // -0 and +0 compare equal
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// dynamic shared memory: uint32 keys[cache_elems] (cache_elems = 0 -> keys are re-read from global)
__global__ void __launch_bounds__(kSelectThreads)
select_kernel(Shape sh, const float* __restrict__ scores, const int32_t* __restrict__ budgets,
              const int32_t* __restrict__ offsets, int32_t* __restrict__ kept_idx, int cache_elems,
              uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint32_t keys_smem[];
  __shared__ uint32_t hist[256];
  __shared__ uint32_t sh_prefix, sh_remaining;
  __shared__ uint32_t warp_gt[kSelectWarps], warp_eq[kSelectWarps];

  const int s = blockIdx.x;
  const int r = s / sh.Hkv, hk = s % sh.Hkv;
  const int p0 = sh.prompt_cu[r], N = sh.prompt_cu[r + 1] - p0;
  const int out0 = offsets[s];
  int k = budgets[s];
  if (k > N) { k = N; if (threadIdx.x == 0) atomicOr(status, (uint32_t)MASKKV_FLAG_BOUNDS); }
  if (k <= 0) return;
  const float* seg = scores + (long long)hk * sh.sumN + p0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (k == N) {                                          // nothing to evict
    for (int j = tid; j < N; j += kSelectThreads) kept_idx[out0 + j] = j;
    return;
  }
  const bool cached = N <= cache_elems;
  if (cached) {
    for (int j = tid; j < N; j += kSelectThreads) keys_smem[j] = order_key(seg[j]);
    __syncthreads();
  }
  auto key_at = [&](int j) -> uint32_t { return cached ? keys_smem[j] : order_key(__ldg(seg + j)); };

  // --- k-th largest key: 4 passes over 8-bit digits, most significant first ---
  uint32_t prefix = 0, have_mask = 0, remaining = (uint32_t)k;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int b = tid; b < 256; b += kSelectThreads) hist[b] = 0;
    __syncthreads();
    for (int j0 = 0; j0 < N; j0 += kSelectThreads) {
      const int j = j0 + tid;
      const bool in = j < N;
      const uint32_t key = in ? key_at(j) : 0u;
      const bool match = in && ((key & have_mask) == prefix);
      const uint32_t digit = (key >> shift) & 0xffu;
      // aggregate equal digits inside the warp so that a crowded bin costs one atomic per warp
      const uint32_t active = __ballot_sync(0xffffffffu, match);
      if (match) {
        const uint32_t peers = __match_any_sync(active, digit);
        if (lane == (31 - __clz(peers))) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
      }
    }
    __syncthreads();
    if (warp == 0) {
      // lane owns digits [8*lane, 8*lane+8); suffix sums from the top digit down
      uint32_t c[8], mine = 0;
#pragma unroll
      for (int t = 0; t < 8; ++t) { c[t] = hist[lane * 8 + t]; mine += c[t]; }
      uint32_t above = mine;                             // inclusive suffix sum over lanes >= lane
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, above, o);
        if (lane + o < 32) above += v;
      }
      above -= mine;                                     // keys with a digit in a higher lane
      uint32_t acc = above;
#pragma unroll
      for (int t = 7; t >= 0; --t) {
        if (acc < remaining && acc + c[t] >= remaining) {  // the k-th largest falls in this digit
          sh_prefix = prefix | ((uint32_t)(lane * 8 + t) << shift);
          sh_remaining = remaining - acc;
        }
        acc += c[t];
      }
    }
    __syncthreads();
    prefix = sh_prefix;
    remaining = sh_remaining;
    have_mask |= 0xffu << shift;
    __syncthreads();
  }
  // prefix = threshold key; `remaining` ties at the threshold are kept, lowest indices first.
  const uint32_t thr = prefix;

  // --- emit in ascending index order: warp w owns [w*span, (w+1)*span) ---
  const int span = ((N + kSelectWarps - 1) / kSelectWarps + 31) & ~31;
  const int wb = min(warp * span, N), we = min(wb + span, N);
  uint32_t n_gt = 0, n_eq = 0;
  for (int j0 = wb; j0 < we; j0 += 32) {
    const int j = j0 + lane;
    const uint32_t key = j < we ? key_at(j) : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, j < we && key > thr));
    n_eq += __popc(__ballot_sync(0xffffffffu, j < we && key == thr));
  }
  if (lane == 0) { warp_gt[warp] = n_gt; warp_eq[warp] = n_eq; }
  __syncthreads();
  uint32_t eq_before = 0, out_before = 0;                // ties / outputs in lower-index warps
  for (int w2 = 0; w2 < warp; ++w2) {
    const uint32_t e2 = warp_eq[w2];
    const uint32_t take = eq_before >= remaining ? 0u : min(e2, remaining - eq_before);
    out_before += warp_gt[w2] + take;
    eq_before += e2;
  }
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int j0 = wb; j0 < we; j0 += 32) {
    const int j = j0 + lane;
    const uint32_t key = j < we ? key_at(j) : 0u;
    const bool gt = j < we && key > thr;
    const bool eq = j < we && key == thr;
    const uint32_t eq_bal = __ballot_sync(0xffffffffu, eq);
    const bool take = gt || (eq && eq_before + __popc(eq_bal & lt_mask) < remaining);
    const uint32_t take_bal = __ballot_sync(0xffffffffu, take);
    if (take) kept_idx[out0 + out_before + __popc(take_bal & lt_mask)] = j;
    out_before += __popc(take_bal);
    eq_before += __popc(eq_bal);
  }
}

}  // namespace mkv

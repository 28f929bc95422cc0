// Gather of the kept K/V rows into the ragged per-head cache: a pure byte copy, eight consecutive kept
// rows per warp and step, 16 bytes per lane per access (K row on the lower half-warp, V row on the
// upper one when a row is 256 bytes).  Bound by HBM; the source rows are scattered 256-byte pieces
// (one DRAM row each), the destination is contiguous.
#pragma once

#include "common.cuh"

namespace mkv {

constexpr int kCompactThreads = 256;
constexpr int kCompactBlocksPerSm = 8;                 // grid cap: about what is resident at once; the blocks loop

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

constexpr int kCompactRows = 8;                         // consecutive output rows a warp moves per step
constexpr int kCompactSmemSegments = 2048;             // offsets[] is staged in shared memory up to this many segments

// row_bytes = d * sizeof(T); strides in bytes.  grid-stride over the rows in use (offsets[S], read on the device).
// PP = 16-byte pieces per lane per row (K row + V row): 1 up to 256-byte rows, 2 for 512-byte rows.
// A warp takes kCompactRows consecutive output rows per step: lane u reads the index of row u and finds its segment (the
// lanes search side by side), the source addresses are handed round by shuffles, then all row pieces of all rows are
// requested before the first one is stored - 4 KB (8 KB) in flight per warp, one dependent chain per eight rows.
template <int PP>
__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(Shape sh, int row_bytes, long long ts_bytes, long long hs_bytes, const unsigned char* __restrict__ kp,
               const unsigned char* __restrict__ vp, const int32_t* __restrict__ kept_idx,
               const int32_t* __restrict__ offsets, long long capacity, unsigned char* __restrict__ kc,
               unsigned char* __restrict__ vc, uint32_t* __restrict__ status) {
  __shared__ int32_t off_s[kCompactSmemSegments + 1];
  __shared__ int32_t pcu_s[kCompactSmemSegments + 1];
  const int S = sh.R * sh.Hkv;
  const bool staged = S <= kCompactSmemSegments;        // the search below then runs out of shared memory
  pdl_launch_dependents();
  pdl_wait();
  if (staged) {
    for (int e = threadIdx.x; e <= S; e += kCompactThreads) off_s[e] = offsets[e];
    for (int e = threadIdx.x; e <= sh.R; e += kCompactThreads) pcu_s[e] = sh.prompt_cu[e];
    __syncthreads();
  }
  const int32_t* off = staged ? off_s : offsets;
  const int32_t* pcu = staged ? pcu_s : sh.prompt_cu;
  long long total = off[S];
  if (total > capacity) total = capacity;
  const int lane = threadIdx.x & 31;
  const int warps_per_block = kCompactThreads / 32;
  const int vec_per_row = row_bytes / 16;               // 16-byte pieces per row (8, 16 or 32)
  const int pieces = 2 * vec_per_row;                   // K row then V row
  const long long warp_id = (long long)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  const long long warps_total = (long long)gridDim.x * warps_per_block;
  for (long long t0 = warp_id * kCompactRows; t0 < total; t0 += warps_total * kCompactRows) {
    // lane u < kCompactRows: source offset of output row t0 + u (-1: no such row, or a bad index that is never followed)
    long long my_src = -1;
    if (lane < kCompactRows && t0 + lane < total) {
      const int j = __ldg(kept_idx + t0 + lane);
      const int s = find_request(off, S, (int)(t0 + lane));   // segment that owns the output row
      const int r = s / sh.Hkv, hk = s % sh.Hkv;
      const int p0 = pcu[r], N = pcu[r + 1] - p0;
      if (j < 0 || j >= N) atomicOr(status, (uint32_t)MASKKV_FLAG_BOUNDS);
      else my_src = (long long)(p0 + j) * ts_bytes + (long long)hk * hs_bytes;
    }
    uint4 v[kCompactRows][PP];
    long long src[kCompactRows];
#pragma unroll
    for (int u = 0; u < kCompactRows; ++u) src[u] = __shfl_sync(0xffffffffu, my_src, u);
#pragma unroll
    for (int u = 0; u < kCompactRows; ++u) {
#pragma unroll
      for (int c = 0; c < PP; ++c) {
        const int e = lane + 32 * c;
        if (src[u] < 0 || e >= pieces) continue;
        const bool is_v = e >= vec_per_row;
        const int o16 = (is_v ? e - vec_per_row : e) * 16;
        v[u][c] = ld_stream(reinterpret_cast<const uint4*>((is_v ? vp : kp) + src[u] + o16));
      }
    }
#pragma unroll
    for (int u = 0; u < kCompactRows; ++u) {
#pragma unroll
      for (int c = 0; c < PP; ++c) {
        const int e = lane + 32 * c;
        if (src[u] < 0 || e >= pieces) continue;
        const bool is_v = e >= vec_per_row;
        const int o16 = (is_v ? e - vec_per_row : e) * 16;
        *reinterpret_cast<uint4*>((is_v ? vc : kc) + (t0 + u) * row_bytes + o16) = v[u][c];
      }
    }
  }
}

}  // namespace mkv

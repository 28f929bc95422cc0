// Top-k eviction (Eq. 16): an exact radix select per (request, head) segment.
//
// One block per segment.  The segment's scores are turned into order-preserving 32-bit keys and
// (when they fit) staged once in shared memory; three histogram passes (11 + 11 + 10 bits) then find
// the k-th largest key exactly, and a last sweep emits the kept indices in ascending order, ties at the
// threshold going to the lowest indices.  Each warp owns a contiguous index range and walks it 32
// consecutive elements at a time, so ranks inside a step come from a ballot and shared-memory
// accesses are conflict-free.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace mkv {

constexpr int kSelectThreads = 1024;
constexpr int kSelectWarps = kSelectThreads / 32;
constexpr int kSelectStaticSmem = 10240;   // upper bound of the kernel's static shared memory (histogram, partials)

// Larger float <=> larger key; NaN maps to 0 (below every number, -inf included).
__device__ __forceinline__ uint32_t order_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;
  if (u == 0x80000000u) u = 0u;                          // -0 and +0 compare equal
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Finds the digit in which the `remaining`-th largest matching key falls, given the histogram of that digit
// (at most 2048 bins; thread t of a THREADS-wide block owns 2048/THREADS consecutive bins).  Returns through
// shared memory: the digit, and how many keys of that digit are still wanted.
template <int THREADS>
__device__ __forceinline__ void find_digit(const uint32_t* hist, int bins, uint32_t remaining, uint32_t* warp_tot,
                                           uint32_t* out_digit, uint32_t* out_remaining) {
  constexpr int BPT = 2048 / THREADS;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t c[BPT], mine = 0;
#pragma unroll
  for (int t = 0; t < BPT; ++t) { c[t] = BPT * tid + t < bins ? hist[BPT * tid + t] : 0u; mine += c[t]; }
  uint32_t suf = mine;                                   // inclusive suffix sum inside the warp (higher lanes = higher digits)
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_down_sync(0xffffffffu, suf, o);
    if (lane + o < 32) suf += v;
  }
  if (lane == 0) warp_tot[warp] = suf;
  __syncthreads();
  uint32_t above = suf - mine;                           // keys with a higher digit
  for (int w2 = warp + 1; w2 < THREADS / 32; ++w2) above += warp_tot[w2];
#pragma unroll
  for (int t = BPT - 1; t >= 0; --t) {                   // highest digit first
    if (above < remaining && above + c[t] >= remaining) { *out_digit = BPT * tid + t; *out_remaining = remaining - above; }
    above += c[t];
  }
  __syncthreads();
}

// Register-resident, four-CTA variant for segments of at most kSelectRegKeys scores.  A thread-block cluster of
// four CTAs shares one segment: CTA q, warp w, lane l keeps key i of index ((q*16 + w)*16 + i)*32 + l in a
// register.  Each CTA histograms its own keys; the four histograms are summed through distributed shared
// memory, so every CTA derives the same digit.  Only the first radix pass looks at every key: the keys that
// fall into its threshold bin are copied to a per-CTA candidate list; every CTA then collects all four lists
// and finishes the search on its own (the lists are short unless the scores are nearly all equal).  The emit sweep visits only the 32-key rows that hold a kept key.  The work is integer issue
// slots, which is why it is spread over four SMs per segment.
constexpr int kSelectCluster = 4;
constexpr int kSelectRegThreads = 512;
constexpr int kSelectRegWarps = kSelectRegThreads / 32;
constexpr int kSelectKeysPerThread = 16;
constexpr int kSelectCandCap = kSelectRegThreads * kSelectKeysPerThread;   // candidate list a CTA holds: its own keys at most, or all CTAs' when they fit
constexpr int kSelectRankMax = 256;                     // candidate lists up to this length are ranked by counting
constexpr int kSelectRegKeys = kSelectCluster * kSelectRegThreads * kSelectKeysPerThread;

// Sum over the cluster of 4 consecutive histogram bins owned by this thread.
__device__ __forceinline__ void cluster_bins(cooperative_groups::cluster_group& cluster, uint32_t* hist, int tid, uint32_t* c) {
  c[0] = c[1] = c[2] = c[3] = 0u;
#pragma unroll
  for (int q = 0; q < kSelectCluster; ++q) {
    const uint4 v = *reinterpret_cast<const uint4*>(cluster.map_shared_rank(hist, q) + 4 * tid);
    c[0] += v.x; c[1] += v.y; c[2] += v.z; c[3] += v.w;
  }
}

// Digit search on cluster-summed counts (thread t owns bins 4t..4t+3); every CTA computes the same answer.
__device__ __forceinline__ void find_digit_counts(const uint32_t* c, uint32_t remaining, uint32_t* warp_tot,
                                                  uint32_t* out_digit, uint32_t* out_remaining) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t mine = (c[0] + c[1]) + (c[2] + c[3]);
  uint32_t suf = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_down_sync(0xffffffffu, suf, o);
    if (lane + o < 32) suf += v;
  }
  if (lane == 0) warp_tot[warp] = suf;
  __syncthreads();
  uint32_t above = suf - mine;
  for (int w2 = warp + 1; w2 < kSelectRegWarps; ++w2) above += warp_tot[w2];
#pragma unroll
  for (int t = 3; t >= 0; --t) {
    if (above < remaining && above + c[t] >= remaining) { *out_digit = 4 * tid + t; *out_remaining = remaining - above; }
    above += c[t];
  }
  __syncthreads();
}

// grid = 4 * segments (cluster of 4 per segment); dynamic shared memory: uint32 cand[kSelectCandCap].
// BLOCKS = CTAs per SM the register budget allows: 1 (94 registers, the fastest single chain: one layer's 32 segments
// all run at once) or 2 (64 registers, twice the segments in flight: batches).
template <int BLOCKS>
__global__ void __cluster_dims__(kSelectCluster, 1, 1) __launch_bounds__(kSelectRegThreads, BLOCKS)
select_kernel_reg(Shape sh, const float* __restrict__ scores, const int32_t* __restrict__ budgets,
                  const int32_t* __restrict__ offsets, int32_t* __restrict__ kept_idx, uint32_t* __restrict__ status) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) uint32_t cand[];
  __shared__ __align__(16) uint32_t hist[2048];
  __shared__ uint32_t sh_digit, sh_remaining, sh_ncand;
  __shared__ uint32_t warp_gt[kSelectRegWarps], warp_eq[kSelectRegWarps], warp_tot[kSelectRegWarps];
  __shared__ uint32_t and_or[2];                         // this CTA's (AND, OR) of its keys, read by the peers
  __shared__ uint32_t gt_eq[2];                          // this CTA's (above, at) threshold counts, read by the peers: a pair of
                                                         // its own, because with all keys equal no cluster barrier lies between a
                                                         // peer's read of and_or and this CTA's write of its counts

  const int s = blockIdx.x / kSelectCluster;
  const int q = (int)cluster.block_rank();
  const int r = s / sh.Hkv, hk = s % sh.Hkv;
  pdl_launch_dependents();
  pdl_wait();
  const int p0 = sh.prompt_cu[r], N = sh.prompt_cu[r + 1] - p0;
  const int out0 = offsets[s];
  int k = budgets[s];
  if (k > N) { k = N; if (threadIdx.x == 0 && q == 0) atomicOr(status, (uint32_t)MASKKV_FLAG_BOUNDS); }
  if (k <= 0) return;                                    // uniform over the cluster
  const float* seg = scores + (long long)hk * sh.sumN + p0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (k == N) {                                          // nothing to evict (uniform over the cluster)
    for (int j = q * kSelectRegThreads + tid; j < N; j += kSelectCluster * kSelectRegThreads) kept_idx[out0 + j] = j;
    return;
  }

  // Warp (q, warp) owns a contiguous, ascending run of keys (the emit step relies on that), `n_rows` rows of 32: the runs
  // are sized to the segment, so a short segment is still spread over all 64 warps of the cluster.
  const int n_rows = min(kSelectKeysPerThread, (N + 32 * kSelectCluster * kSelectRegWarps - 1) / (32 * kSelectCluster * kSelectRegWarps));
  const int jbase = (q * kSelectRegWarps + warp) * (32 * n_rows) + lane;
  uint32_t key[kSelectKeysPerThread];
#pragma unroll
  for (int i = 0; i < kSelectKeysPerThread; ++i) {        // all loads first: the whole segment is in flight at once
    const int j = jbase + i * 32;
    key[i] = (i < n_rows && j < N) ? __float_as_uint(__ldg(seg + j)) : 0u;
  }
  uint32_t vmask = 0u;                                   // bit i: key i exists
  uint32_t k_and = 0xffffffffu, k_or = 0u;
#pragma unroll
  for (int i = 0; i < kSelectKeysPerThread; ++i) {
    key[i] = order_key(__uint_as_float(key[i]));
    if (i < n_rows && jbase + i * 32 < N) { vmask |= 1u << i; k_and &= key[i]; k_or |= key[i]; }
  }
  k_and = __reduce_and_sync(0xffffffffu, k_and);
  k_or = __reduce_or_sync(0xffffffffu, k_or);
  if (tid < 32) { warp_gt[tid & (kSelectRegWarps - 1)] = 0xffffffffu; warp_eq[tid & (kSelectRegWarps - 1)] = 0u; }
  for (int b2 = tid; b2 < 2048; b2 += kSelectRegThreads) hist[b2] = 0;
  if (tid == 0) sh_ncand = 0;
  __syncthreads();
  if (lane == 0) { warp_gt[warp] = k_and; warp_eq[warp] = k_or; }
  __syncthreads();
  if (warp == 0) {
    k_and = __reduce_and_sync(0xffffffffu, warp_gt[lane & (kSelectRegWarps - 1)]);
    k_or = __reduce_or_sync(0xffffffffu, warp_eq[lane & (kSelectRegWarps - 1)]);
    if (lane == 0) { and_or[0] = k_and; and_or[1] = k_or; }
  }
  cluster.sync();
  k_and = 0xffffffffu; k_or = 0u;
#pragma unroll
  for (int c = 0; c < kSelectCluster; ++c) {
    const uint32_t* peer = cluster.map_shared_rank(and_or, c);
    k_and &= peer[0];
    k_or |= peer[1];
  }
  // Leading bits on which every key agrees carry no order information: the radix starts below them.
  const int common = __clz(k_and ^ k_or);                // 32 when all keys are equal
  int bits_left = 32 - common;
  uint32_t have_mask = common == 0 ? 0u : (common == 32 ? 0xffffffffu : ~(0xffffffffu >> common));
  uint32_t prefix = k_and & have_mask;
  uint32_t remaining = (uint32_t)k;
  uint32_t cnt4[4];

  if (bits_left > 0) {
    // first pass: every key (all of them match the common prefix)
    const int width = bits_left >= 11 ? 11 : bits_left;
    const int shift = bits_left - width;
    const uint32_t dmask = (1u << width) - 1u;
#pragma unroll
    for (int i = 0; i < kSelectKeysPerThread; ++i)
      if ((vmask >> i) & 1u) atomicAdd(&hist[(key[i] >> shift) & dmask], 1u);
    cluster.sync();
    cluster_bins(cluster, hist, tid, cnt4);
    find_digit_counts(cnt4, remaining, warp_tot, &sh_digit, &sh_remaining);
    prefix |= sh_digit << shift;
    remaining = sh_remaining;
    have_mask |= dmask << shift;
    bits_left = shift;
    if (bits_left > 0) {
      // the keys of the threshold bin become this CTA's candidate list
#pragma unroll
      for (int i = 0; i < kSelectKeysPerThread; ++i) {
        const bool m = ((vmask >> i) & 1u) && (key[i] & have_mask) == prefix;
        const uint32_t bal = __ballot_sync(0xffffffffu, m);
        if (bal) {
          uint32_t pos = 0;
          if (lane == 0) pos = atomicAdd(&sh_ncand, (uint32_t)__popc(bal));
          pos = __shfl_sync(0xffffffffu, pos, 0);
          if (m) cand[pos + __popc(bal & ((1u << lane) - 1u))] = key[i];
        }
      }
    }
    cluster.sync();                                      // peers are done with this CTA's histogram; candidates are complete
    if (bits_left > 0) {
      // Every CTA appends its peers' candidates to its own (through distributed shared memory) and finishes the
      // search on its own: the same list in a different order gives the same histogram, hence the same threshold.
      int ncand = (int)sh_ncand;
      const int own = ncand;
      int n_peer[kSelectCluster], total = own;
#pragma unroll
      for (int c = 1; c < kSelectCluster; ++c) {
        n_peer[c] = (int)*cluster.map_shared_rank(&sh_ncand, (q + c) & (kSelectCluster - 1));
        total += n_peer[c];
      }
      if (total > kSelectCandCap) {
        // Too many keys share the threshold bin (nearly equal scores) for every CTA to hold them all: the lists stay
        // where they are and the remaining digits are found like the first one, with histograms summed over the cluster.
#pragma unroll 1
        while (bits_left > 0) {
          const int w2 = bits_left >= 11 ? 11 : bits_left;
          const int sh2 = bits_left - w2;
          const uint32_t dm2 = (1u << w2) - 1u;
          for (int b2 = tid; b2 < 2048; b2 += kSelectRegThreads) hist[b2] = 0;
          __syncthreads();
          for (int t = tid; t < own; t += kSelectRegThreads) {
            const uint32_t c = cand[t];
            if ((c & have_mask) == prefix) atomicAdd(&hist[(c >> sh2) & dm2], 1u);
          }
          cluster.sync();
          cluster_bins(cluster, hist, tid, cnt4);
          find_digit_counts(cnt4, remaining, warp_tot, &sh_digit, &sh_remaining);
          prefix |= sh_digit << sh2;
          remaining = sh_remaining;
          have_mask |= dm2 << sh2;
          bits_left = sh2;
          cluster.sync();                                  // every peer has read this histogram before it is cleared again
        }
      } else {
#pragma unroll
        for (int c = 1; c < kSelectCluster; ++c) {
          const uint32_t* src = cluster.map_shared_rank(cand, (q + c) & (kSelectCluster - 1));
          for (int t = tid; t < n_peer[c]; t += kSelectRegThreads) cand[ncand + t] = src[t];
          ncand += n_peer[c];
        }
      }
      if (bits_left > 0 && ncand <= kSelectRankMax) {
        // A short list (the usual case: the threshold bin of an 11-bit digit over 32k keys holds tens of keys): the
        // threshold is the candidate with fewer than `remaining` candidates above it and at least `remaining` at or
        // above it - one pass of broadcast reads instead of two more histogram passes.
        __syncthreads();                                   // the gathered list is complete
        if (tid < ncand) {
          const uint32_t mine = cand[tid];
          uint32_t gt = 0, ge = 0;
          for (int u = 0; u < ncand; ++u) {
            const uint32_t c = cand[u];
            gt += c > mine;
            ge += c >= mine;
          }
          if (gt < remaining && remaining <= ge) { sh_digit = mine; sh_remaining = remaining - gt; }   // equal keys write equal values
        }
        __syncthreads();
        prefix = sh_digit;
        remaining = sh_remaining;
        bits_left = 0;
      }
#pragma unroll 1
      while (bits_left > 0) {
        const int w2 = bits_left >= 11 ? 11 : bits_left;
        const int sh2 = bits_left - w2;
        const uint32_t dm2 = (1u << w2) - 1u;
        for (int b2 = tid; b2 < 2048; b2 += kSelectRegThreads) hist[b2] = 0;
        __syncthreads();
        for (int t = tid; t < ncand; t += kSelectRegThreads) {
          const uint32_t c = cand[t];
          if ((c & have_mask) == prefix) atomicAdd(&hist[(c >> sh2) & dm2], 1u);
        }
        __syncthreads();
        find_digit<kSelectRegThreads>(hist, 2048, remaining, warp_tot, &sh_digit, &sh_remaining);
        prefix |= sh_digit << sh2;
        remaining = sh_remaining;
        have_mask |= dm2 << sh2;
        bits_left = sh2;
      }
    }
  }
  const uint32_t thr = prefix;                           // threshold key; `remaining` ties are kept, lowest indices first

  uint32_t gt_mask = 0u, eq_mask = 0u;
#pragma unroll
  for (int i = 0; i < kSelectKeysPerThread; ++i) {
    if ((vmask >> i) & 1u) {
      if (key[i] > thr) gt_mask |= 1u << i;
      if (key[i] == thr) eq_mask |= 1u << i;
    }
  }
  const uint32_t n_gt = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(gt_mask));
  const uint32_t n_eq = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(eq_mask));
  __syncthreads();                                       // warp_gt / warp_eq are reused
  if (lane == 0) { warp_gt[warp] = n_gt; warp_eq[warp] = n_eq; }
  __syncthreads();
  if (warp == 0) {                                       // this CTA's totals, for the CTAs after it
    const uint32_t g = __reduce_add_sync(0xffffffffu, lane < kSelectRegWarps ? warp_gt[lane] : 0u);
    const uint32_t e = __reduce_add_sync(0xffffffffu, lane < kSelectRegWarps ? warp_eq[lane] : 0u);
    if (lane == 0) { gt_eq[0] = g; gt_eq[1] = e; }
  }
  cluster.sync();
  // ties / outputs that precede this warp: the lower CTAs as wholes, then the lower warps of this CTA
  uint32_t eq_before = 0, out_before = 0;
  {
    uint32_t pg[kSelectCluster], pe[kSelectCluster];
#pragma unroll
    for (int c = 0; c < kSelectCluster; ++c) {
      const uint32_t* peer = cluster.map_shared_rank(gt_eq, c);
      pg[c] = c < q ? peer[0] : 0u;
      pe[c] = c < q ? peer[1] : 0u;
    }
#pragma unroll
    for (int c = 0; c < kSelectCluster; ++c) {
      const uint32_t take = eq_before >= remaining ? 0u : min(pe[c], remaining - eq_before);
      out_before += pg[c] + take;
      eq_before += pe[c];
    }
    for (int w2 = 0; w2 < warp; ++w2) {
      const uint32_t e2 = warp_eq[w2];
      const uint32_t take = eq_before >= remaining ? 0u : min(e2, remaining - eq_before);
      out_before += warp_gt[w2] + take;
      eq_before += e2;
    }
  }
  cluster.barrier_arrive();                              // done reading the peers' shared memory (waited for at the end)
  // rows of this warp that hold a key at or above the threshold, lowest row first
  uint32_t rows = __reduce_or_sync(0xffffffffu, gt_mask | eq_mask);
  const uint32_t lt_mask = (1u << lane) - 1u;
  while (rows) {
    const int i = __ffs((int)rows) - 1;
    rows &= rows - 1;
    const bool gt = (gt_mask >> i) & 1u, eq = (eq_mask >> i) & 1u;
    const uint32_t eq_bal = __ballot_sync(0xffffffffu, eq);
    const bool take = gt || (eq && eq_before + __popc(eq_bal & lt_mask) < remaining);
    const uint32_t take_bal = __ballot_sync(0xffffffffu, take);
    if (take) kept_idx[out0 + out_before + __popc(take_bal & lt_mask)] = jbase + i * 32;
    out_before += __popc(take_bal);
    eq_before += __popc(eq_bal);
  }
  cluster.barrier_wait();                                // no CTA leaves while a peer may still read its shared memory
}

// One CTA per segment with the keys in REGISTERS, for batches of segments of up to kSelectBlockKeys scores (the launch
// over all (layer, head) segments of a model, a ragged serving batch): 1024 threads hold 32 keys each, so after the one
// coalesced read of the segment no pass touches memory again - a pass costs two to four instructions per key instead of
// an index computation, a bounds test and a shared-memory load on top.  Warp w owns the contiguous keys
// [w * 32 * n_rows, (w + 1) * 32 * n_rows), row i of a thread is key jbase + 32 * i, so ranks inside a row come from a
// ballot and the output is ascending.
// The k-th largest key is found inside a window [lo, lo + range] of key values that starts as [smallest key, largest
// key] and shrinks by a factor of up to 2048 per pass: digit = (key - lo) >> shift with the smallest shift that maps
// the window onto 2048 bins.  Unlike a digit of fixed bit positions this spreads the keys over the bins whatever
// power of two the scores happen to straddle (few populated bins would serialise the shared-memory atomics).  After a
// pass either the threshold bin's keys are gathered into a short list (ranked by counting, or by further digits on the
// list) or - when that bin holds more than the list - the next digit is taken on the registers again.  One emit pass.
// Blocks take the requests in order of falling length, so a ragged batch ends with its short segments.
constexpr int kSelectBlockThreads = 1024;
constexpr int kSelectBlockWarps = kSelectBlockThreads / 32;
constexpr int kSelectBlockRows = 32;                     // keys per thread
constexpr int kSelectBlockKeys = kSelectBlockThreads * kSelectBlockRows;   // 32768
constexpr int kSelectBlockCand = 4096;

// order_key in five instructions: x + 0 turns -0 into +0 (and keeps everything else, NaN included)
__device__ __forceinline__ uint32_t order_key_lean(float f) {
  const uint32_t u = __float_as_uint(f + 0.f);
  const uint32_t key = u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);
  return (u & 0x7fffffffu) > 0x7f800000u ? 0u : key;
}

struct SelectBlockShared {
  uint32_t hist[2048];
  uint32_t cand[kSelectBlockCand];
  uint32_t digit, remaining, ncand;
  uint32_t warp_a[kSelectBlockWarps], warp_b[kSelectBlockWarps], warp_tot[kSelectBlockWarps];
};

// FULL: every thread holds kSelectBlockRows keys (N = kSelectBlockKeys), so no row needs a validity test.
template <bool FULL>
__device__ __forceinline__ void select_block_body(SelectBlockShared& sm, const float* __restrict__ seg, int N, int k,
                                                  int32_t* __restrict__ kept) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_rows = FULL ? kSelectBlockRows : min(kSelectBlockRows, (N + 32 * kSelectBlockWarps - 1) / (32 * kSelectBlockWarps));
  const int jbase = warp * (32 * n_rows) + lane;
  const int nv = FULL ? kSelectBlockRows : max(0, min(n_rows, (N - jbase + 31) >> 5));   // rows 0 .. nv-1 hold a key
  uint32_t key[kSelectBlockRows];
#pragma unroll
  for (int i = 0; i < kSelectBlockRows; ++i) key[i] = (FULL || i < nv) ? __float_as_uint(__ldg(seg + jbase + i * 32)) : 0u;   // all loads first
  // Scores are sums of softmax weights: +0 or positive and finite unless the inputs were not.  The bit patterns of such
  // floats already order like the numbers, so they serve as keys as they are; one signed minimum and one unsigned
  // maximum per key find the window and tell whether every score is of that kind (a negative number, -0 or a NaN
  // shows as a negative minimum or a maximum above +inf).  Otherwise the keys are transformed and the window taken again.
  int32_t s_min = 0x7fffffff;
  uint32_t k_max = 0u;
#pragma unroll
  for (int i = 0; i < kSelectBlockRows; ++i)
    if (FULL || i < nv) { s_min = min(s_min, (int32_t)key[i]); k_max = max(k_max, key[i]); }
  s_min = __reduce_min_sync(0xffffffffu, s_min);
  k_max = __reduce_max_sync(0xffffffffu, k_max);
  if (lane == 0) { sm.warp_a[warp] = (uint32_t)s_min; sm.warp_b[warp] = k_max; }
  for (int b = tid; b < 2048; b += kSelectBlockThreads) sm.hist[b] = 0;
  if (tid == 0) sm.ncand = 0;
  __syncthreads();
  s_min = __reduce_min_sync(0xffffffffu, (int32_t)sm.warp_a[lane]);
  k_max = __reduce_max_sync(0xffffffffu, sm.warp_b[lane]);
  uint32_t lo = (uint32_t)s_min;
  __syncthreads();                                       // warp_a / warp_b are reused below
  if (s_min < 0 || k_max > 0x7f800000u) {                // block-uniform: some score is negative, -0 or NaN
    uint32_t k_min = 0xffffffffu;
    k_max = 0u;
#pragma unroll
    for (int i = 0; i < kSelectBlockRows; ++i) {
      key[i] = order_key_lean(__uint_as_float(key[i]));
      if (FULL || i < nv) { k_min = min(k_min, key[i]); k_max = max(k_max, key[i]); }
    }
    k_min = __reduce_min_sync(0xffffffffu, k_min);
    k_max = __reduce_max_sync(0xffffffffu, k_max);
    if (lane == 0) { sm.warp_a[warp] = k_min; sm.warp_b[warp] = k_max; }
    __syncthreads();
    lo = __reduce_min_sync(0xffffffffu, sm.warp_a[lane]);
    k_max = __reduce_max_sync(0xffffffffu, sm.warp_b[lane]);
    __syncthreads();
  }
  uint32_t range = k_max - lo;                           // 0 when all keys are equal
  uint32_t remaining = (uint32_t)k;

  int ncand = -1;                                        // >= 0: the search continues on cand[0 .. ncand)
  bool first = true;                                     // every key lies inside the window
#pragma unroll 1
  while (range > 0 && ncand < 0) {                       // digits on the registers
    const int shift = max(0, 21 - __clz(range));         // (range >> shift) < 2048
    if (first) {
#pragma unroll
      for (int i = 0; i < kSelectBlockRows; ++i)
        if (FULL || i < nv) atomicAdd(&sm.hist[(key[i] - lo) >> shift], 1u);
    } else {
#pragma unroll
      for (int i = 0; i < kSelectBlockRows; ++i) {
        const uint32_t d = key[i] - lo;
        if ((FULL || i < nv) && d <= range) atomicAdd(&sm.hist[d >> shift], 1u);
      }
    }
    first = false;
    __syncthreads();
    find_digit<kSelectBlockThreads>(sm.hist, 2048, remaining, sm.warp_tot, &sm.digit, &sm.remaining);
    const uint32_t in_bin = sm.hist[sm.digit];           // keys that share the threshold digit
    const uint32_t step = sm.digit << shift;
    lo += step;
    range = min(range - step, (uint32_t)((1ull << shift) - 1ull));
    remaining = sm.remaining;
    __syncthreads();                                     // everyone has read the histogram and the digit
    if (range > 0) {
      if (in_bin <= (uint32_t)kSelectBlockCand) {
        // few enough: gather them (a thread rarely holds more than one) and finish on the list
#pragma unroll
        for (int i = 0; i < kSelectBlockRows; ++i)
          if ((FULL || i < nv) && key[i] - lo <= range) sm.cand[atomicAdd(&sm.ncand, 1u)] = key[i];
        __syncthreads();
        ncand = (int)sm.ncand;
      } else {
        for (int b = tid; b < 2048; b += kSelectBlockThreads) sm.hist[b] = 0;
        __syncthreads();
      }
    }
  }
  if (range > 0 && ncand <= kSelectRankMax) {
    // a short list: the threshold is the candidate with fewer than `remaining` candidates above it and at least
    // `remaining` at or above it
    if (tid < ncand) {
      const uint32_t mine = sm.cand[tid];
      uint32_t gt = 0, ge = 0;
      for (int u = 0; u < ncand; ++u) {
        const uint32_t c = sm.cand[u];
        gt += c > mine;
        ge += c >= mine;
      }
      if (gt < remaining && remaining <= ge) { sm.digit = mine; sm.remaining = remaining - gt; }   // equal keys write equal values
    }
    __syncthreads();
    lo = sm.digit;
    remaining = sm.remaining;
    range = 0;
  }
#pragma unroll 1
  while (range > 0) {                                    // further digits on the list
    const int shift = max(0, 21 - __clz(range));
    __syncthreads();
    for (int b = tid; b < 2048; b += kSelectBlockThreads) sm.hist[b] = 0;
    __syncthreads();
    for (int j = tid; j < ncand; j += kSelectBlockThreads) {
      const uint32_t d = sm.cand[j] - lo;
      if (d <= range) atomicAdd(&sm.hist[d >> shift], 1u);
    }
    __syncthreads();
    find_digit<kSelectBlockThreads>(sm.hist, 2048, remaining, sm.warp_tot, &sm.digit, &sm.remaining);
    const uint32_t step = sm.digit << shift;
    lo += step;
    range = min(range - step, (uint32_t)((1ull << shift) - 1ull));
    remaining = sm.remaining;
  }
  const uint32_t thr = lo;                               // threshold key; `remaining` ties are kept, lowest indices first

  // --- emit in ascending index order ---
  // Usually the ties at the threshold are all kept (one key there, one wanted): then "at or above the threshold" is the
  // whole test.  Only when more keys tie than are wanted are the ties told apart from the keys above.
  uint32_t gt_mask = 0u, eq_mask = 0u;
#pragma unroll
  for (int i = 0; i < kSelectBlockRows; ++i)
    if ((FULL || i < nv) && key[i] >= thr) gt_mask |= 1u << i;
  {
    const uint32_t n_ge = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(gt_mask));
    if (lane == 0) sm.warp_a[warp] = n_ge;
    __syncthreads();
    const uint32_t total = __reduce_add_sync(0xffffffffu, sm.warp_a[lane]);
    if (total != (uint32_t)k) {                          // block-uniform: more ties than wanted
      gt_mask = 0u;
#pragma unroll
      for (int i = 0; i < kSelectBlockRows; ++i) {
        if (FULL || i < nv) {
          if (key[i] > thr) gt_mask |= 1u << i;
          if (key[i] == thr) eq_mask |= 1u << i;
        }
      }
    } else {
      remaining = 0;                                     // no key counts as a tie
    }
    __syncthreads();                                     // warp_a is written again below
  }
  const uint32_t n_gt = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(gt_mask));
  const uint32_t n_eq = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(eq_mask));
  if (lane == 0) { sm.warp_a[warp] = n_gt; sm.warp_b[warp] = n_eq; }
  __syncthreads();
  // ties / outputs in lower-index warps: lane l looks at warp l, a warp scan gives the totals before this warp
  uint32_t eq_before = 0, out_before = 0;
  {
    const uint32_t g = sm.warp_a[lane], e = sm.warp_b[lane];
    uint32_t e_incl = e;                                 // inclusive prefix of the tie counts
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, e_incl, o);
      if (lane >= o) e_incl += v;
    }
    const uint32_t e_excl = e_incl - e;
    const uint32_t take = e_excl >= remaining ? 0u : min(e, remaining - e_excl);
    uint32_t o_incl = g + take;                          // outputs of warp l
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, o_incl, o);
      if (lane >= o) o_incl += v;
    }
    eq_before = __shfl_sync(0xffffffffu, e_excl, warp);
    out_before = __shfl_sync(0xffffffffu, o_incl - (g + take), warp);
  }
  uint32_t rows = __reduce_or_sync(0xffffffffu, gt_mask | eq_mask);
  const uint32_t lt_mask = (1u << lane) - 1u;
  while (rows) {                                         // rows of this warp that hold a key at or above the threshold
    const int i = __ffs((int)rows) - 1;
    rows &= rows - 1;
    const bool gt = (gt_mask >> i) & 1u, eq = (eq_mask >> i) & 1u;
    const uint32_t eq_bal = __ballot_sync(0xffffffffu, eq);
    const bool take = gt || (eq && eq_before + __popc(eq_bal & lt_mask) < remaining);
    const uint32_t take_bal = __ballot_sync(0xffffffffu, take);
    if (take) kept[out_before + __popc(take_bal & lt_mask)] = jbase + i * 32;
    out_before += __popc(take_bal);
    eq_before += __popc(eq_bal);
  }
}

__global__ void __launch_bounds__(kSelectBlockThreads, 1)
select_kernel_block(Shape sh, const float* __restrict__ scores, const int32_t* __restrict__ budgets,
                    const int32_t* __restrict__ offsets, int32_t* __restrict__ kept_idx, uint32_t* __restrict__ status) {
  __shared__ __align__(16) SelectBlockShared sm;
  const int tid = threadIdx.x;
  pdl_launch_dependents();
  pdl_wait();
  if (tid == 0) sm.digit = 0u;
  __syncthreads();
  for (int t = tid; t < sh.R; t += kSelectBlockThreads) {  // the request that is number blockIdx / H_kv by falling length
    const int nt = sh.prompt_cu[t + 1] - sh.prompt_cu[t];
    int rank = 0;
    for (int u = 0; u < sh.R; ++u) {
      const int nu = sh.prompt_cu[u + 1] - sh.prompt_cu[u];
      rank += (nu > nt || (nu == nt && u < t)) ? 1 : 0;
    }
    if (rank == (int)blockIdx.x / sh.Hkv) sm.digit = (uint32_t)t;
  }
  __syncthreads();
  const int r = (int)sm.digit, hk = (int)blockIdx.x % sh.Hkv;
  const int s = r * sh.Hkv + hk;
  const int p0 = sh.prompt_cu[r], N = sh.prompt_cu[r + 1] - p0;
  const int out0 = offsets[s];
  int k = budgets[s];
  if (k > N) { k = N; if (tid == 0) atomicOr(status, (uint32_t)MASKKV_FLAG_BOUNDS); }
  if (k <= 0) return;
  const float* seg = scores + (long long)hk * sh.sumN + p0;
  if (k == N) {                                          // nothing to evict
    for (int j = tid; j < N; j += kSelectBlockThreads) kept_idx[out0 + j] = j;
    return;
  }
  __syncthreads();                                       // sm.digit has been read by everyone
  if (N == kSelectBlockKeys) select_block_body<true>(sm, seg, N, k, kept_idx + out0);
  else select_block_body<false>(sm, seg, N, k, kept_idx + out0);
}

// One CTA per segment, for batches of segments: the keys are staged in shared memory once and every pass over them
// runs eight rows of 32 keys at a time per warp with the loads ahead of the uses (the cluster kernel above is built
// for the latency of one layer's few segments; with hundreds of segments its clusters queue up in waves that each
// wait on cluster barriers).  Passes over all keys: staging (with the common prefix), the first 11-bit histogram,
// the copy of the threshold bin's keys to a candidate list, and the two emit sweeps; the remaining digits are found
// on the candidate list (ranked by counting when short).  Warp w owns the contiguous keys [w*span, (w+1)*span).
// dynamic shared memory: uint32 keys[n_cache] followed by uint32 cand[kSelectCtaCand]; N <= n_cache.
constexpr int kSelectCtaCand = 4096;

__global__ void __launch_bounds__(kSelectThreads)
select_kernel_cta(Shape sh, const float* __restrict__ scores, const int32_t* __restrict__ budgets,
                  const int32_t* __restrict__ offsets, int32_t* __restrict__ kept_idx, int n_cache,
                  uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint32_t keys_smem[];
  uint32_t* cand = keys_smem + n_cache;
  __shared__ uint32_t hist[2048];
  __shared__ uint32_t sh_digit, sh_remaining, sh_ncand;
  __shared__ uint32_t warp_gt[kSelectWarps], warp_eq[kSelectWarps], warp_tot[kSelectWarps];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_dependents();
  pdl_wait();
  // Blocks are handed out in index order, so the longest prompts go first: block b takes the request that is
  // number b / H_kv when the requests are sorted by falling length (ties by index) - a ragged batch then ends with
  // its short segments instead of with a last wave of long ones.
  if (tid == 0) sh_digit = 0u;
  __syncthreads();
  for (int t = tid; t < sh.R; t += kSelectThreads) {
    const int nt = sh.prompt_cu[t + 1] - sh.prompt_cu[t];
    int rank = 0;
    for (int u = 0; u < sh.R; ++u) {
      const int nu = sh.prompt_cu[u + 1] - sh.prompt_cu[u];
      rank += (nu > nt || (nu == nt && u < t)) ? 1 : 0;
    }
    if (rank == (int)blockIdx.x / sh.Hkv) sh_digit = (uint32_t)t;
  }
  __syncthreads();
  const int r = (int)sh_digit, hk = (int)blockIdx.x % sh.Hkv;
  const int s = r * sh.Hkv + hk;
  const int p0 = sh.prompt_cu[r], N = sh.prompt_cu[r + 1] - p0;
  const int out0 = offsets[s];
  int k = budgets[s];
  if (k > N) { k = N; if (threadIdx.x == 0) atomicOr(status, (uint32_t)MASKKV_FLAG_BOUNDS); }
  if (k <= 0) return;
  const float* seg = scores + (long long)hk * sh.sumN + p0;
  if (k == N) {                                          // nothing to evict
    for (int j = tid; j < N; j += kSelectThreads) kept_idx[out0 + j] = j;
    return;
  }
  __syncthreads();                                       // sh_digit is reused below

  // --- stage the keys and find the bits they all share ---
  uint32_t k_and = 0xffffffffu, k_or = 0u;
  auto stage = [&](int j, float f) {
    const uint32_t key = order_key(f);
    keys_smem[j] = key;
    k_and &= key;
    k_or |= key;
  };
  {
    const int head = min(N, (int)((4 - (((long long)hk * sh.sumN + p0) & 3)) & 3));   // scalars up to the first aligned score
    const int n4 = (N - head) >> 2;
    const float4* seg4 = reinterpret_cast<const float4*>(seg + head);
    for (int j = tid; j < head; j += kSelectThreads) stage(j, seg[j]);
    for (int i0 = 0; i0 < n4; i0 += 8 * kSelectThreads) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * kSelectThreads + tid;
        if (i < n4) v[u] = __ldg(seg4 + i);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * kSelectThreads + tid;
        if (i < n4) {
          const int j = head + 4 * i;
          stage(j, v[u].x); stage(j + 1, v[u].y); stage(j + 2, v[u].z); stage(j + 3, v[u].w);
        }
      }
    }
    for (int j = head + 4 * n4 + tid; j < N; j += kSelectThreads) stage(j, seg[j]);
  }
  k_and = __reduce_and_sync(0xffffffffu, k_and);
  k_or = __reduce_or_sync(0xffffffffu, k_or);
  if (lane == 0) { warp_gt[warp] = k_and; warp_eq[warp] = k_or; }
  for (int b = tid; b < 2048; b += kSelectThreads) hist[b] = 0;
  if (tid == 0) sh_ncand = 0;
  __syncthreads();
  k_and = __reduce_and_sync(0xffffffffu, warp_gt[lane]);
  k_or = __reduce_or_sync(0xffffffffu, warp_eq[lane]);
  const int common = __clz(k_and ^ k_or);                // 32 when all keys are equal
  int bits_left = 32 - common;
  uint32_t have_mask = common == 0 ? 0u : (common == 32 ? 0xffffffffu : ~(0xffffffffu >> common));
  uint32_t prefix = k_and & have_mask;
  uint32_t remaining = (uint32_t)k;

  // this warp's keys: rows of 32 consecutive keys, eight rows per step
  const int span = ((N + kSelectWarps - 1) / kSelectWarps + 31) & ~31;
  const int wb = min(warp * span, N), we = min(wb + span, N);

  int ncand = -1;                                        // -1: the candidate list is not in use (all keys still count)
  if (bits_left > 0) {
    // first digit: every key matches the common prefix
    const int width = bits_left >= 11 ? 11 : bits_left;
    const int shift = bits_left - width;
    const uint32_t dmask = (1u << width) - 1u;
    for (int j0 = wb; j0 < we; j0 += 256) {
      uint32_t kk[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) { const int j = j0 + 32 * u + lane; kk[u] = j < we ? keys_smem[j] : 0u; }
#pragma unroll
      for (int u = 0; u < 8; ++u) { const int j = j0 + 32 * u + lane; if (j < we) atomicAdd(&hist[(kk[u] >> shift) & dmask], 1u); }
    }
    __syncthreads();
    find_digit<kSelectThreads>(hist, 1 << width, remaining, warp_tot, &sh_digit, &sh_remaining);
    prefix |= sh_digit << shift;
    remaining = sh_remaining;
    have_mask |= dmask << shift;
    bits_left = shift;
    if (bits_left > 0) {
      // the keys of the threshold bin become the candidate list (appended per row with one atomic per warp)
      for (int j0 = wb; j0 < we; j0 += 256) {
        uint32_t kk[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) { const int j = j0 + 32 * u + lane; kk[u] = j < we ? keys_smem[j] : 0u; }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int j = j0 + 32 * u + lane;
          const bool m = j < we && (kk[u] & have_mask) == prefix;
          const uint32_t bal = __ballot_sync(0xffffffffu, m);
          if (bal) {
            uint32_t pos = 0;
            if (lane == 0) pos = atomicAdd(&sh_ncand, (uint32_t)__popc(bal));
            pos = __shfl_sync(0xffffffffu, pos, 0);
            const uint32_t at = pos + __popc(bal & ((1u << lane) - 1u));
            if (m && at < (uint32_t)kSelectCtaCand) cand[at] = kk[u];
          }
        }
      }
      __syncthreads();
      ncand = (int)sh_ncand;
      if (ncand > kSelectCtaCand) ncand = -1;            // too many nearly equal scores: keep working on all keys
    }
  }
  if (bits_left > 0 && ncand >= 0 && ncand <= kSelectRankMax) {
    // a short list: the threshold is the candidate with fewer than `remaining` candidates above it and at least
    // `remaining` at or above it
    if (tid < ncand) {
      const uint32_t mine = cand[tid];
      uint32_t gt = 0, ge = 0;
      for (int u = 0; u < ncand; ++u) {
        const uint32_t c = cand[u];
        gt += c > mine;
        ge += c >= mine;
      }
      if (gt < remaining && remaining <= ge) { sh_digit = mine; sh_remaining = remaining - gt; }   // equal keys write equal values
    }
    __syncthreads();
    prefix = sh_digit;
    remaining = sh_remaining;
    bits_left = 0;
  }
#pragma unroll 1
  while (bits_left > 0) {                                // further digits: on the list, or on all keys when it overflowed
    const int width = bits_left >= 11 ? 11 : bits_left;
    const int shift = bits_left - width, bins = 1 << width;
    const uint32_t dmask = (uint32_t)(bins - 1);
    __syncthreads();
    for (int b = tid; b < bins; b += kSelectThreads) hist[b] = 0;
    __syncthreads();
    const uint32_t* src = ncand >= 0 ? cand : keys_smem;
    const int n_src = ncand >= 0 ? ncand : N;
    for (int j = tid; j < n_src; j += kSelectThreads) {
      const uint32_t key = src[j];
      if ((key & have_mask) == prefix) atomicAdd(&hist[(key >> shift) & dmask], 1u);
    }
    __syncthreads();
    find_digit<kSelectThreads>(hist, bins, remaining, warp_tot, &sh_digit, &sh_remaining);
    prefix |= sh_digit << shift;
    remaining = sh_remaining;
    have_mask |= dmask << shift;
    bits_left = shift;
  }
  const uint32_t thr = prefix;                           // threshold key; `remaining` ties are kept, lowest indices first

  // --- emit in ascending index order ---
  uint32_t n_gt = 0, n_eq = 0;
  for (int j0 = wb; j0 < we; j0 += 256) {
    uint32_t kk[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) { const int j = j0 + 32 * u + lane; kk[u] = j < we ? keys_smem[j] : 0u; }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int j = j0 + 32 * u + lane;
      n_gt += (j < we && kk[u] > thr) ? 1u : 0u;
      n_eq += (j < we && kk[u] == thr) ? 1u : 0u;
    }
  }
  n_gt = __reduce_add_sync(0xffffffffu, n_gt);
  n_eq = __reduce_add_sync(0xffffffffu, n_eq);
  __syncthreads();                                       // warp_gt / warp_eq are reused
  if (lane == 0) { warp_gt[warp] = n_gt; warp_eq[warp] = n_eq; }
  __syncthreads();
  uint32_t eq_before = 0, out_before = 0;                // ties / outputs in lower-index warps
  for (int w2 = 0; w2 < warp; ++w2) {
    const uint32_t e2 = warp_eq[w2];
    const uint32_t take = eq_before >= remaining ? 0u : min(e2, remaining - eq_before);
    out_before += warp_gt[w2] + take;
    eq_before += e2;
  }
  if (n_gt + n_eq == 0) return;                          // nothing of this warp's range is kept
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int j0 = wb; j0 < we; j0 += 256) {
    uint32_t kk[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) { const int j = j0 + 32 * u + lane; kk[u] = j < we ? keys_smem[j] : 0u; }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int j = j0 + 32 * u + lane;
      const bool gt = j < we && kk[u] > thr;
      const bool eq = j < we && kk[u] == thr;
      const uint32_t any_bal = __ballot_sync(0xffffffffu, gt || eq);
      if (any_bal == 0u) continue;                       // warp-uniform: most rows hold no kept key
      const uint32_t eq_bal = __ballot_sync(0xffffffffu, eq);
      const bool take = gt || (eq && eq_before + __popc(eq_bal & lt_mask) < remaining);
      const uint32_t take_bal = __ballot_sync(0xffffffffu, take);
      if (take) kept_idx[out0 + out_before + __popc(take_bal & lt_mask)] = j;
      out_before += __popc(take_bal);
      eq_before += __popc(eq_bal);
    }
  }
}

// dynamic shared memory: uint32 keys[cache_elems] (cache_elems = 0 -> keys are re-read from global)
__global__ void __launch_bounds__(kSelectThreads)
select_kernel(Shape sh, const float* __restrict__ scores, const int32_t* __restrict__ budgets,
              const int32_t* __restrict__ offsets, int32_t* __restrict__ kept_idx, int cache_elems,
              uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint32_t keys_smem[];
  __shared__ uint32_t hist[2048];
  __shared__ uint32_t sh_digit, sh_remaining;
  __shared__ uint32_t warp_gt[kSelectWarps], warp_eq[kSelectWarps], warp_tot[kSelectWarps];

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
  auto key_at = [&](int j) -> uint32_t { return cached ? keys_smem[j] : order_key(__ldg(seg + j)); };

  // --- stage the keys and find the bits they all share ---
  uint32_t k_and = 0xffffffffu, k_or = 0u;
  auto stage = [&](int j, float f) {
    const uint32_t key = order_key(f);
    if (cached) keys_smem[j] = key;
    k_and &= key;
    k_or |= key;
  };
  {
    // 16-byte loads, eight in flight per thread: the whole segment is requested before the first key is used
    const int head = min(N, (int)((4 - (((long long)hk * sh.sumN + p0) & 3)) & 3));   // scalars up to the first aligned score
    const int n4 = (N - head) >> 2;
    const float4* seg4 = reinterpret_cast<const float4*>(seg + head);
    for (int j = tid; j < head; j += kSelectThreads) stage(j, seg[j]);
    for (int i0 = 0; i0 < n4; i0 += 8 * kSelectThreads) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * kSelectThreads + tid;
        if (i < n4) v[u] = __ldg(seg4 + i);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * kSelectThreads + tid;
        if (i < n4) {
          const int j = head + 4 * i;
          stage(j, v[u].x); stage(j + 1, v[u].y); stage(j + 2, v[u].z); stage(j + 3, v[u].w);
        }
      }
    }
    for (int j = head + 4 * n4 + tid; j < N; j += kSelectThreads) stage(j, seg[j]);
  }
  k_and = __reduce_and_sync(0xffffffffu, k_and);
  k_or = __reduce_or_sync(0xffffffffu, k_or);
  if (lane == 0) { warp_gt[warp] = k_and; warp_eq[warp] = k_or; }
  __syncthreads();
  k_and = warp_gt[lane];
  k_or = warp_eq[lane];
  k_and = __reduce_and_sync(0xffffffffu, k_and);
  k_or = __reduce_or_sync(0xffffffffu, k_or);
  __syncthreads();
  // Leading bits on which every key agrees carry no order information: the radix starts below them, so the
  // first digit is spread over its bins however narrow the range of the scores is.
  const int common = __clz(k_and ^ k_or);                // 32 when all keys are equal
  int bits_left = 32 - common;
  uint32_t prefix = common == 0 ? 0u : (k_and & ~(0xffffffffu >> common));
  uint32_t have_mask = common == 0 ? 0u : ~(0xffffffffu >> common);
  if (common == 32) { prefix = k_and; have_mask = 0xffffffffu; }
  uint32_t remaining = (uint32_t)k;

  // --- k-th largest key: passes over 11-bit digits (the last one takes what is left), most significant first ---
#pragma unroll 1
  while (bits_left > 0) {
    const int width = bits_left >= 11 ? 11 : bits_left;
    const int shift = bits_left - width, bins = 1 << width;
    for (int b = tid; b < bins; b += kSelectThreads) hist[b] = 0;
    __syncthreads();
    for (int j = tid; j < N; j += kSelectThreads) {
      const uint32_t key = key_at(j);
      if ((key & have_mask) == prefix) atomicAdd(&hist[(key >> shift) & (uint32_t)(bins - 1)], 1u);
    }
    __syncthreads();
    find_digit<kSelectThreads>(hist, bins, remaining, warp_tot, &sh_digit, &sh_remaining);
    prefix |= sh_digit << shift;
    remaining = sh_remaining;
    have_mask |= (uint32_t)(bins - 1) << shift;
    bits_left = shift;
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
  if (n_gt + n_eq == 0) return;                          // nothing of this warp's range is kept
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

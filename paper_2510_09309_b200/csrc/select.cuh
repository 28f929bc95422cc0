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
  if (THREADS == 1024) {                                 // 32 warps: lane l looks at warp l
    above += __reduce_add_sync(0xffffffffu, lane > warp ? warp_tot[lane] : 0u);
  } else {
    for (int w2 = warp + 1; w2 < THREADS / 32; ++w2) above += warp_tot[w2];
  }
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

#ifdef MASKKV_DBG_SELECT_CLOCK
__device__ unsigned int g_sel_prints = 0;
#define SEL_STAMP(n) do { if (blockIdx.x == 5 && threadIdx.x == 0) st_[n] = clock64(); } while (0)
#else
#define SEL_STAMP(n) do { } while (0)
#endif
struct SelectBlockShared {
  uint32_t hist[2048];
  uint32_t cand[kSelectBlockCand];
  int32_t cand_idx[kSelectBlockCand];                     // indices of the listed keys (sampled short cut)
  uint32_t digit, remaining, ncand;
  uint32_t warp_a[kSelectBlockWarps], warp_b[kSelectBlockWarps], warp_tot[kSelectBlockWarps];
};

// FULL: every thread holds kSelectBlockRows keys (N = kSelectBlockKeys), so no row needs a validity test.
// Short cut for the usual case (few keys wanted out of many): one key per thread serves as a sample; a histogram of the
// samples gives a bound `lo` that - unless the samples mislead - lies below the k-th largest key with few keys above it.
// One pass over the registers collects the keys at or above `lo` (key and index, in ascending index order) in shared
// memory; the k-th largest is then found on that list and the kept set is a compaction of the list.  Two passes over
// the registers less than the full search, and none of its 32 histogram updates per thread.  Returns false, having
// written nothing, when the short cut does not apply (a sample that is negative, -0 or NaN; too many keys wanted; fewer
// than k or more than the list holds at or above `lo`): the caller then runs the full search on the same registers.
template <bool FULL, class Load, class Release>
__device__ __forceinline__ bool select_block_sampled(SelectBlockShared& sm, const uint32_t (&key)[kSelectBlockRows], int nv, int jbase,
                                                     int N, int k, int32_t* __restrict__ kept, Load load, Release release) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt_mask = (1u << lane) - 1u;
  const bool has = FULL || nv > 0;
#ifdef MASKKV_DBG_SELECT_CLOCK
  long long st_[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#endif
  SEL_STAMP(0);
  const uint32_t smp = key[0];
  {
    const uint32_t mn = __reduce_min_sync(0xffffffffu, has ? smp : 0xffffffffu);
    const uint32_t mx = __reduce_max_sync(0xffffffffu, has ? smp : 0u);
    const uint32_t ns = (uint32_t)__popc(__ballot_sync(0xffffffffu, has));
    if (lane == 0) { sm.warp_a[warp] = mn; sm.warp_b[warp] = mx; sm.warp_tot[warp] = ns; }
  }
  for (int b = tid; b < 2048; b += kSelectBlockThreads) sm.hist[b] = 0;
  __syncthreads();
  uint32_t lo = __reduce_min_sync(0xffffffffu, sm.warp_a[lane]);
  const uint32_t s_max = __reduce_max_sync(0xffffffffu, sm.warp_b[lane]);
  const uint32_t n_s = __reduce_add_sync(0xffffffffu, sm.warp_tot[lane]);
  __syncthreads();                                       // the per-warp slots are written again below
  if (s_max > 0x7f800000u) return false;                 // raw bits do not order like the numbers
  const float mu = (float)k * (float)n_s / (float)N;     // samples expected above the k-th largest key
  const uint32_t r_lo = (uint32_t)(mu + 5.f * sqrtf(mu) + 4.f);
  if (r_lo >= n_s || (long long)r_lo * N > 3072LL * n_s) return false;
  if (s_max > lo) {
    const int shift = max(0, 21 - __clz(s_max - lo));
    if (has) atomicAdd(&sm.hist[(smp - lo) >> shift], 1u);
    __syncthreads();
    find_digit<kSelectBlockThreads>(sm.hist, 2048, r_lo, sm.warp_tot, &sm.digit, &sm.remaining);
    lo += sm.digit << shift;
  }
  SEL_STAMP(1);
  // keys at or above lo: bit i of `mask` = row i of this thread
  uint32_t mask = 0u;
#pragma unroll
  for (int i = 0; i < kSelectBlockRows; ++i)
    if ((FULL || i < nv) && key[i] >= lo) mask |= 1u << i;
  // Transpose the warp's 32 x 32 bits: lane i then holds the ballot of row i, so the list positions (ascending index:
  // warps own consecutive index ranges, rows ascend, lanes ascend) come from one scan over the rows instead of a ballot
  // per row.  The histogram is free by now: warp w keeps its 32 ballots and 32 row offsets in hist[64 w ...].
  uint32_t bal = mask;
#pragma unroll
  for (int sft = 16; sft >= 1; sft >>= 1) {
    const uint32_t keep = sft == 16 ? 0x0000ffffu : sft == 8 ? 0x00ff00ffu : sft == 4 ? 0x0f0f0f0fu : sft == 2 ? 0x33333333u : 0x55555555u;
    const uint32_t other = __shfl_xor_sync(0xffffffffu, bal, sft);
    bal = (lane & sft) ? (((other >> sft) & keep) | (bal & ~keep)) : ((bal & keep) | ((other & keep) << sft));
  }
  __syncthreads();                                       // every thread is done with the histogram of the samples
  uint32_t C, pos;
  {
    const uint32_t cnt = (uint32_t)__popc(bal);
    uint32_t incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t u = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += u;
    }
    sm.hist[warp * 64 + lane] = bal;
    sm.hist[warp * 64 + 32 + lane] = incl - cnt;
    if (lane == 31) sm.warp_a[warp] = incl;
    __syncthreads();
    const uint32_t v = sm.warp_a[lane];
    uint32_t w_incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t u = __shfl_up_sync(0xffffffffu, w_incl, o);
      if (lane >= o) w_incl += u;
    }
    C = __shfl_sync(0xffffffffu, w_incl, 31);
    pos = __shfl_sync(0xffffffffu, w_incl - v, warp);
  }
  SEL_STAMP(2);
  if (C < (uint32_t)k || C > (uint32_t)kSelectBlockCand) { __syncthreads(); return false; }
  // a thread rarely holds more than one listed key: it lists the indices, and the keys are read back by list position
  // (the segment is still in the staging buffer or in the caches) - indexing the registers by a run-time row would not do
  for (uint32_t m = mask; m != 0u; m &= m - 1u) {
    const int i = __ffs((int)m) - 1;
    sm.cand_idx[pos + sm.hist[warp * 64 + 32 + i] + __popc(sm.hist[warp * 64 + i] & lt_mask)] = jbase + i * 32;
  }
  __syncthreads();
  {
    uint32_t l_max = 0u;
    for (int j = tid; j < (int)C; j += kSelectBlockThreads) {
      const uint32_t c = load(sm.cand_idx[j]);
      sm.cand[j] = c;
      l_max = max(l_max, c);
    }
    l_max = __reduce_max_sync(0xffffffffu, l_max);
    if (lane == 0) sm.warp_b[warp] = l_max;
  }
  __syncthreads();
  release();                                             // the segment's copy is no longer needed
  const uint32_t k_max = __reduce_max_sync(0xffffffffu, sm.warp_b[lane]);
  __syncthreads();
  if (k_max > 0x7f800000u) return false;                 // a negative score, -0 or a NaN somewhere in the segment
  const int ncand = (int)C;
  SEL_STAMP(3);
  uint32_t range = k_max - lo, remaining = (uint32_t)k;
  // rank by counting on a short list of keys: the wanted key has fewer than `remaining` keys above it and at least
  // `remaining` at or above it
  auto rank_short = [&](const uint32_t* list, int n) {
    if (tid < n) {
      const uint32_t mine_k = list[tid];
      uint32_t gt = 0, ge = 0;
      for (int u = 0; u < n; ++u) {
        const uint32_t c = list[u];
        gt += c > mine_k;
        ge += c >= mine_k;
      }
      if (gt < remaining && remaining <= ge) { sm.digit = mine_k; sm.remaining = remaining - gt; }   // equal keys write equal values
    }
    __syncthreads();
    lo = sm.digit;
    remaining = sm.remaining;
    range = 0;
  };
  if (range > 0 && ncand <= kSelectRankMax) rank_short(sm.cand, ncand);
#pragma unroll 1
  while (range > 0) {                                    // digits on the list, within the window [lo, lo + range]
    const int shift = max(0, 21 - __clz(range));
    __syncthreads();
    for (int b = tid; b < 2048; b += kSelectBlockThreads) sm.hist[b] = 0;
    if (tid == 0) sm.ncand = 0;
    __syncthreads();
    for (int j = tid; j < ncand; j += kSelectBlockThreads) {
      const uint32_t d = sm.cand[j] - lo;
      if (d <= range) atomicAdd(&sm.hist[d >> shift], 1u);
    }
    __syncthreads();
    find_digit<kSelectBlockThreads>(sm.hist, 2048, remaining, sm.warp_tot, &sm.digit, &sm.remaining);
    const uint32_t in_bin = sm.hist[sm.digit];
    const uint32_t step = sm.digit << shift;
    lo += step;
    range = min(range - step, (uint32_t)((1ull << shift) - 1ull));
    remaining = sm.remaining;
    __syncthreads();                                     // everyone has read the histogram and the digit
    if (range > 0 && in_bin <= (uint32_t)kSelectRankMax) {
      // the few keys of the threshold bin, copied over the histogram and ranked by counting
      for (int j = tid; j < ncand; j += kSelectBlockThreads) {
        const uint32_t c = sm.cand[j];
        if (c - lo <= range) sm.hist[atomicAdd(&sm.ncand, 1u)] = c;
      }
      __syncthreads();
      rank_short(sm.hist, (int)sm.ncand);
    }
  }
  const uint32_t thr = lo;                               // the k-th largest key; `remaining` keys equal to it are kept, lowest indices first
  SEL_STAMP(4);
  // the kept set: a compaction of the list
  uint32_t carry_out = 0, carry_eq = 0;
#pragma unroll 1
  for (int base = 0; base < ncand; base += kSelectBlockThreads) {
    const int j = base + tid;
    const uint32_t kj = j < ncand ? sm.cand[j] : 0u;
    const bool gt = j < ncand && kj > thr, eq = j < ncand && kj == thr;
    const uint32_t gt_bal = __ballot_sync(0xffffffffu, gt), eq_bal = __ballot_sync(0xffffffffu, eq);
    __syncthreads();                                     // the per-warp slots may still be read (previous round, searches above)
    if (lane == 0) { sm.warp_a[warp] = __popc(gt_bal); sm.warp_b[warp] = __popc(eq_bal); }
    __syncthreads();
    const uint32_t g = sm.warp_a[lane], e = sm.warp_b[lane];
    uint32_t e_incl = e;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, e_incl, o);
      if (lane >= o) e_incl += v;
    }
    const uint32_t e_excl = carry_eq + e_incl - e;
    const uint32_t take_w = e_excl >= remaining ? 0u : min(e, remaining - e_excl);
    uint32_t o_incl = g + take_w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, o_incl, o);
      if (lane >= o) o_incl += v;
    }
    const uint32_t eq_before = __shfl_sync(0xffffffffu, e_excl, warp);
    const uint32_t out_before = carry_out + __shfl_sync(0xffffffffu, o_incl - (g + take_w), warp);
    const bool take = gt || (eq && eq_before + __popc(eq_bal & lt_mask) < remaining);
    const uint32_t take_bal = __ballot_sync(0xffffffffu, take);
    if (take) kept[out_before + __popc(take_bal & lt_mask)] = sm.cand_idx[j];
    carry_eq += __shfl_sync(0xffffffffu, e_incl, 31);
    carry_out += __shfl_sync(0xffffffffu, o_incl, 31);
  }
#ifdef MASKKV_DBG_SELECT_CLOCK
  SEL_STAMP(5);
  if (blockIdx.x == 5 && threadIdx.x == 0 && g_sel_prints < 6u)
    printf("sampled: sample %lld count %lld gather %lld threshold %lld emit %lld ncand %d k %d\n", st_[1] - st_[0], st_[2] - st_[1], st_[3] - st_[2], st_[4] - st_[3], st_[5] - st_[4], ncand, k);
#endif
  return true;
}

// `load(j)` returns the bits of score j of the segment; `loaded()` runs (all threads) once every key is in registers.
template <bool FULL, class Load, class Loaded>
__device__ __forceinline__ void select_block_body(SelectBlockShared& sm, Load load, Loaded loaded, int N, int k,
                                                  int32_t* __restrict__ kept) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_rows = FULL ? kSelectBlockRows : min(kSelectBlockRows, (N + 32 * kSelectBlockWarps - 1) / (32 * kSelectBlockWarps));
  const int jbase = warp * (32 * n_rows) + lane;
  const int nv = FULL ? kSelectBlockRows : max(0, min(n_rows, (N - jbase + 31) >> 5));   // rows 0 .. nv-1 hold a key
  uint32_t key[kSelectBlockRows];
#ifdef MASKKV_DBG_SELECT_CLOCK
  long long st_[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#endif
  SEL_STAMP(0);
#pragma unroll
  for (int i = 0; i < kSelectBlockRows; ++i) key[i] = (FULL || i < nv) ? load(jbase + i * 32) : 0u;   // all loads first
  bool released = false;
  auto release = [&] { if (!released) { loaded(); released = true; } };   // block-uniform
  SEL_STAMP(1);
#ifndef MASKKV_SELECT_NO_SAMPLING
  if (select_block_sampled<FULL>(sm, key, nv, jbase, N, k, kept, load, release)) {
#ifdef MASKKV_DBG_SELECT_CLOCK
    SEL_STAMP(6);
    if (blockIdx.x == 5 && threadIdx.x == 0 && atomicAdd(&g_sel_prints, 1u) < 6u) printf("select sampled path: %lld cycles after the load\n", st_[6] - st_[1]);
#endif
    return;
  }
  __syncthreads();                                       // the short cut's shared state is reused by the full search
#endif
  release();
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
  SEL_STAMP(2);

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
    SEL_STAMP(3);
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
  SEL_STAMP(4);
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
  SEL_STAMP(5);

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
#ifdef MASKKV_DBG_SELECT_CLOCK
  SEL_STAMP(6);
  if (blockIdx.x == 5 && threadIdx.x == 0 && atomicAdd(&g_sel_prints, 1u) < 6u)
    printf("select phases (cycles): load %lld window %lld hist %lld digit+gather %lld rank %lld emit %lld ncand %d\n", st_[1] - st_[0],
           st_[2] - st_[1], st_[3] - st_[2], st_[4] - st_[3], st_[5] - st_[4], st_[6] - st_[5], ncand);
#endif
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
  auto load = [&](int j) { return __float_as_uint(__ldg(seg + j)); };
  auto loaded = [] {};
  if (N == kSelectBlockKeys) select_block_body<true>(sm, load, loaded, N, k, kept_idx + out0);
  else select_block_body<false>(sm, load, loaded, N, k, kept_idx + out0);
}

// ---------------------------------------------------------------------------------------------------------------------
// The same selection for launches with more segments than SMs: one persistent CTA per SM takes segments b, b + G, ... of
// the falling-length order, and while it works on one segment the next one's scores arrive in shared memory through ONE
// bulk copy issued by one thread (no per-thread copy instructions: what a per-thread staging of the next segment cost in
// instructions used up what it hid).  The buffer is free again as soon as the keys are in registers, so a single buffer
// gives a whole segment's arithmetic of lead.  The copy moves the 16-byte-aligned middle of the segment; up to three
// scores at either end are fetched with plain loads.  Waits on the copy are bounded (about a second), then the block
// raises MASKKV_FLAG_TIMEOUT and leaves.
__device__ __forceinline__ uint32_t sel_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool sel_mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(sel_smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool sel_mbar_wait(uint64_t* bar, uint32_t parity) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (sel_mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u) {
      unsigned long long now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (t0 == 0) t0 = now;
      else if (now - t0 > 1000000000ull) return false;
    }
  }
}

struct SelectItem { int N, k, out0; const float* seg; };
constexpr int kSelectStreamSmem = (kSelectBlockKeys + 4) * 4;   // dynamic shared memory: the staged scores

__global__ void __launch_bounds__(kSelectBlockThreads, 1)
select_kernel_stream(Shape sh, const float* __restrict__ scores, const int32_t* __restrict__ budgets,
                     const int32_t* __restrict__ offsets, int32_t* __restrict__ kept_idx, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) float stage[];           // kSelectBlockKeys + 4 scores
  __shared__ __align__(16) SelectBlockShared sm;
  __shared__ __align__(8) uint64_t bar;
  __shared__ int item_r;
  const int tid = threadIdx.x, n_items = sh.R * sh.Hkv;
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sel_smem_u32(&bar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  pdl_launch_dependents();
  pdl_wait();
  __syncthreads();

  // segment number `item` of the falling-length order (block-uniform; two barriers)
  auto locate = [&](int item) {
    for (int t = tid; t < sh.R; t += kSelectBlockThreads) {
      const int nt = sh.prompt_cu[t + 1] - sh.prompt_cu[t];
      int rank = 0;
      for (int u = 0; u < sh.R; ++u) {
        const int nu = sh.prompt_cu[u + 1] - sh.prompt_cu[u];
        rank += (nu > nt || (nu == nt && u < t)) ? 1 : 0;
      }
      if (rank == item / sh.Hkv) item_r = t;
    }
    __syncthreads();
    const int r = item_r, hk = item % sh.Hkv, s = r * sh.Hkv + hk;
    __syncthreads();
    SelectItem it;
    const int p0 = sh.prompt_cu[r];
    it.N = sh.prompt_cu[r + 1] - p0;
    it.out0 = offsets[s];
    it.k = budgets[s];
    if (it.k > it.N) { it.k = it.N; if (tid == 0) atomicOr(status, (uint32_t)MASKKV_FLAG_BOUNDS); }
    it.seg = scores + (long long)hk * sh.sumN + p0;
    return it;
  };
  auto staged = [](const SelectItem& it) { return it.k > 0 && it.k < it.N; };
  // score j of the segment lands in stage[mis + j], mis = the segment's offset from a 16-byte boundary in floats
  auto issue = [&](const SelectItem& it) {
    if (!staged(it)) return;
    const int mis = (int)((reinterpret_cast<uintptr_t>(it.seg) & 15u) >> 2);
    const int e0 = min((4 - mis) & 3, it.N);               // scores in front of the first 16-byte boundary
    const int n_mid = (it.N - e0) & ~3;
    float* dst = stage + mis;
    if (tid == 0) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the buffer was last read with ordinary loads
      if (n_mid > 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(sel_smem_u32(&bar)), "r"(n_mid * 4) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(sel_smem_u32(dst + e0)), "l"(it.seg + e0), "r"(n_mid * 4), "r"(sel_smem_u32(&bar)) : "memory");
      } else {
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(sel_smem_u32(&bar)) : "memory");
      }
    } else if (tid >= 32 && tid < 40) {
      const int e = tid - 32;
      const int j = e < 4 ? e : e0 + n_mid + (e - 4);
      if (e < 4 ? e < e0 : j < it.N) dst[j] = __ldg(it.seg + j);
    }
  };

  int item = blockIdx.x;
  if (item >= n_items) return;
  SelectItem cur = locate(item);
  issue(cur);
  uint32_t parity = 0;
  for (;;) {
    const int next = item + (int)gridDim.x;
    const bool have_next = next < n_items;
    SelectItem nxt = cur;
    if (have_next) nxt = locate(next);
    bool next_issued = false;
    if (cur.k >= cur.N && cur.k > 0) {                     // nothing to evict
      for (int j = tid; j < cur.N; j += kSelectBlockThreads) kept_idx[cur.out0 + j] = j;
    } else if (cur.k > 0) {
      const bool ok = sel_mbar_wait(&bar, parity);
      parity ^= 1u;
      if (!__syncthreads_and(ok)) {                        // also orders the edge scores written by other threads
        if (tid == 0) atomicOr(status, (uint32_t)MASKKV_FLAG_TIMEOUT);
        return;
      }
      const float* src = stage + (int)((reinterpret_cast<uintptr_t>(cur.seg) & 15u) >> 2);
      auto load = [&](int j) { return __float_as_uint(src[j]); };
      auto loaded = [&] {
        __syncthreads();                                   // every key is in registers: the buffer is free
        if (have_next) issue(nxt);
        next_issued = true;
      };
      if (cur.N == kSelectBlockKeys) select_block_body<true>(sm, load, loaded, cur.N, cur.k, kept_idx + cur.out0);
      else select_block_body<false>(sm, load, loaded, cur.N, cur.k, kept_idx + cur.out0);
    }
    if (!have_next) break;
    __syncthreads();                                       // the body's shared state is reused by the next segment
    if (!next_issued) issue(nxt);
    item = next;
    cur = nxt;
  }
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

// Mask-voting scores (Eq. 6-7, sums of Eq. 14) for bf16 inputs on the 5th-generation tensor cores.
//
// The logits S = Q K^T are produced tile by tile by tcgen05.mma into tensor memory and consumed there:
// the M x (N+M) weight matrix never exists in shared or global memory.  Column sums need each row's
// final normaliser, so the product is formed twice:
//
//   sweep 1  score_stats_tc   queries on the TMEM lanes (A = 128-query tile, B = 128-key tile): the thread
//                             that owns a lane owns a softmax row and keeps its running (max, sum of exp).
//                             A unit covers 256 queries (two accumulators) x one run of key tiles and
//                             yields one partial per row and CTA; sweep 2 merges the partials into lse_i when it
//                             loads a query block.
//   sweep 2  score_colsum_tc  keys on the TMEM lanes (A = 128-key tile, B = up to 256 queries): the owning
//                             thread reads its key's logits against every query, forms
//                             A_ij = 2^(s_ij*c - lse2_i) and sums over i in a register - the column sum
//                             needs no cross-thread reduction.  It also sums the attention masses; with several
//                             query blocks per KV head a small kernel adds the blocks' column sums.
//
// Both kernels are persistent (one CTA per SM walks an equal, contiguous share of the sweep's tiles, its
// TMA / MMA / epilogue pipelines running on across segment boundaries) and warp-specialised: warp 0 issues TMA loads (4-stage
// ring of key tiles), warp 1 issues the MMAs, warps 2-17 are four epilogue warpgroups - two per
// accumulator, each taking half of its columns - so that every scheduler has four warps of
// exponentials to interleave while the tensor pipe fills the other accumulator.  Tensor memory: 512 columns
// = 2 x 256 (sweep 2) or 4 x 128 (sweep 1).  Both sweeps are bound by the exponential (MUFU) rate.
#include "score_tc.h"

#include "tc_common.cuh"

namespace mkv {
namespace tc {

constexpr int kThreads = 576;          // 18 warps: TMA, MMA, 4 x 4 epilogue
constexpr int kEpiThreadsPerAcc = 256; // two epilogue warpgroups share one accumulator
constexpr int kStages = 4;
constexpr int kTile = 128;             // keys per tile (both sweeps), queries per accumulator (sweep 1)
constexpr int kQBlock = 256;           // queries resident per CTA
constexpr int kColsumPad = 3;          // sweep 2: what entering a new unit costs a CTA, in key tiles (see Walker)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
// Share of the exponentials that runs as a polynomial on the FMA pipes instead of on the special-function unit (16 results
// per clock per SM): this many pairs out of every eight.  Measured on B200 (32k LLaDA layer / 16k Dream layer, whole call):
// sweep 2 with 0 / 2 / 3 / 4 pairs 171.7 / 169.3 / 176.0 / 182.2 us and 162.4 / 157.8 / 161.3 / 169.6 us; sweep 1 with
// 0 / 2 / 3 pairs 171.6 / 176.8 / 176.7 us.  A stand-alone loop of the same epilogue gains 24 % at 3 of 8; inside the
// kernels the sweeps are held by the hand-over of the accumulators and by the key stream as much as by the exponentials,
// so only the small share in sweep 2 pays.  Compile-time switches so that the comparison can be repeated.
#ifndef MASKKV_STATS_POLY
#define MASKKV_STATS_POLY 0
#endif
#ifndef MASKKV_COLSUM_POLY
#define MASKKV_COLSUM_POLY 2
#endif
constexpr int kStatsPolyPairs = MASKKV_STATS_POLY;      // sweep 1, degree 2 (row sums average the error away)
constexpr int kColsumPolyPairs = MASKKV_COLSUM_POLY;
// Measurement switches (off in the library): MASKKV_DBG_NOMATH leaves the epilogues with their tensor-memory loads and
// barrier traffic only, MASKKV_DBG_KSTEPS issues that many of the eight MMA k-steps per tile - together they show what the
// key stream, the products and the accumulator hand-over cost without the exponentials.
#ifndef MASKKV_DBG_KSTEPS
#define MASKKV_DBG_KSTEPS 8
#endif
// Two more timing probes for sweep 2 (both give wrong scores): MASKKV_DBG_RELEASE_AT=c hands the accumulator back to the MMA
// issuer as soon as chunk c of its columns is in registers (0 = three chunks early), MASKKV_DBG_NOTAIL drops everything a
// warp does per tile after its exponentials (exchange of the halves, score stores, mass sums).  Measured on B200 at the 32k
// layer, whole call: 175.0 us as shipped; release at chunk 0 / 1 / 2: 174.8 / 174.8 / 175.4; no tail: 173.2; one MMA k-step
// of eight with all the arithmetic: 164.4.  Neither the hand-over of the accumulators, nor the per-tile tail, nor the
// products hold the sweeps: the epilogue's own instruction stream does (96 registers per thread where the compiler would
// take 150 for sweep 2 and 204 for sweep 1 if it could).
// which pairs of a group of eight go to the polynomial: spread out, so that both units always have work in flight
__host__ __device__ constexpr bool poly_pair(int pair, int n_of_8) {
  return ((pair & 7) + 1) * n_of_8 / 8 > (pair & 7) * n_of_8 / 8;
}

template <int D>
struct Smem {
  static constexpr int kBoxes = D / 64;
  static constexpr int kQBoxBytes = kQBlock * 128;          // one 64-column box of the 256 resident queries
  static constexpr int kQBytes = kBoxes * kQBoxBytes;
  static constexpr int kKBoxBytes = kTile * 128;
  static constexpr int kKBytes = kBoxes * kKBoxBytes;
  static constexpr int kQOff = 0;
  static constexpr int kKOff = kQBytes;
  static constexpr int kC2Off = kKOff + kStages * kKBytes;                 // float [4 warpgroups][2][128] per-query constants
  static constexpr int kS2Off = kC2Off + 4 * kQBlock * 4;                  // float [4 warpgroups][2][128] second constants (polynomial columns)
  static constexpr int kXchOff = kS2Off + 4 * kQBlock * 4;                 // float [2 accumulators][2][128]
  static constexpr int kBarOff = kXchOff + 4 * kTile * 4;                  // mbarriers
  static constexpr int kNumBars = 2 * kStages + 2 + 4 + 4;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;                  // tmem base, abort flag
  static constexpr int kBytes = kMiscOff + 16;
  static constexpr int kDynamic = kBytes + 1024;                           // room to align the base to 1024
};

struct Bars {
  uint64_t* full;     // [kStages]  key tile landed
  uint64_t* empty;    // [kStages]  key tile consumed by the MMAs
  uint64_t* qfull;    // resident queries landed
  uint64_t* qempty;   // resident queries no longer read by any MMA
  uint64_t* tfull;    // [4] accumulator written
  uint64_t* tempty;   // [4] accumulator drained by its epilogue warpgroup
};

__device__ __forceinline__ Bars carve_bars(uint8_t* base, int bar_off) {
  uint64_t* b = reinterpret_cast<uint64_t*>(base + bar_off);
  Bars r;
  r.full = b; r.empty = b + kStages; r.qfull = b + 2 * kStages; r.qempty = r.qfull + 1; r.tfull = r.qempty + 1; r.tempty = r.tfull + 4;
  return r;
}

// After an abandoned wait the producer still owns the TMA copies it has issued: wait (bounded) for the
// most recent ones so that no copy lands in shared memory after the block has exited.
__device__ __forceinline__ void drain_loads(const Bars& bars, int issued) {
  for (int i = max(0, issued - kStages); i < issued; ++i) {
    const int stage = i % kStages, use = i / kStages;
    for (uint32_t it = 0; it < (1u << 20) && !mbar_try_wait(bars.full + stage, use & 1); ++it) __nanosleep(64);
  }
}

__device__ __forceinline__ uint8_t* align_1024(uint8_t* p) {
  return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

// Tile t of request r in the order [prompt tiles ; mask tiles]: which tensor, which token row, how many valid keys.
struct KeyTile { bool prompt; int token; int valid; };
__device__ __forceinline__ KeyTile key_tile(int t, int p0, int N, int l0, int M) {
  const int TP = (N + kTile - 1) / kTile;
  KeyTile k;
  k.prompt = t < TP;
  const int off = (k.prompt ? t : t - TP) * kTile;
  k.token = (k.prompt ? p0 : l0) + off;
  k.valid = min(kTile, (k.prompt ? N : M) - off);
  return k;
}

__device__ __forceinline__ void block_setup(const Bars& bars, int n_acc, uint32_t* tmem_slot, volatile uint32_t* abort_flag) {
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(bars.full + s, 1); mbar_init(bars.empty + s, 1); }
    mbar_init(bars.qfull, 1); mbar_init(bars.qempty, 1);
    for (int b = 0; b < n_acc; ++b) { mbar_init(bars.tfull + b, 1); mbar_init(bars.tempty + b, kEpiThreadsPerAcc); }
    *abort_flag = 0u;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
}

__device__ __forceinline__ void block_teardown(uint32_t tmem_base) {
  tc_fence_before();
  __syncthreads();
  if ((threadIdx.x >> 5) == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

// =====================================================================================================
// Work distribution.  The tiles of a sweep form one flat sequence ordered by (request, group, tile), where a
// group is a (query head, 256-query block) in sweep 1 and a KV head in sweep 2.  CTA c of G takes the
// contiguous share [c*F/G, (c+1)*F/G) of the F tiles - every CTA gets the same number of tiles to within one -
// and walks it one segment (a run of tiles of one group) at a time.  Every role of the CTA runs the same walk.
// =====================================================================================================
// tiles t, t+dir, ..., len of them; unit_start = flat index of the unit's first position in this walk (padding included),
// unit_real = the same without any padding (the index sweep 1's walk gives the unit)
struct Seg { int r, g, t, len, p0, N, l0, M, T, dir; long long unit_start, unit_real; };

// mode of a walk: sweep 1 (groups = query head x 256-query block), sweep 2 with one query block per KV head (groups =
// KV heads), sweep 2 with several (groups = query head x block again; the blocks' column sums meet in a later kernel)
enum { kWalkStats = 0, kWalkColsum = 1, kWalkColsumSplit = 2 };

// `pad`: positions without work put in front of every unit's tiles (sweep 2 only).  Crossing into a new unit costs a CTA
// about as much as `pad` tiles (new queries, the merge of their normalisers, the hand-over of the attention mass), and
// the shares are equal in positions, so a share that contains a unit boundary gets that many tiles fewer.
struct Walker {
  long long f, f_end, base, base_real;   // forward: [f, f_end) still to do; reverse: [f_end, f) still to do, taken from the top
  int r, mode, pad;
  bool reverse;
};

__host__ __device__ __forceinline__ int walk_groups(const Shape& sh, int mode, int M) {
  return M <= 0 ? 0 : (mode == kWalkColsum ? sh.hkn : sh.hkn * sh.g * ((M + kQBlock - 1) / kQBlock));
}
__device__ __forceinline__ int tiles_of(int N, int M) { return (N + kTile - 1) / kTile + (M + kTile - 1) / kTile; }

// Sweep 2 walks every share backwards: it then starts on the tiles sweep 1 read last, which are the ones most
// likely to be still in L2 (the key tensor of a long prompt is larger than L2, so a forward walk would miss all).
__device__ __forceinline__ void walker_init(Walker& w, const Shape& sh, int mode, bool reverse, long long F, int pad = 0) {
  w.mode = mode;
  w.reverse = reverse;
  w.pad = pad;
  const long long lo = (long long)blockIdx.x * F / gridDim.x, hi = (long long)(blockIdx.x + 1) * F / gridDim.x;
  w.base = 0;
  w.base_real = 0;
  w.r = 0;
  if (!reverse) { w.f = lo; w.f_end = hi; return; }        // forward walks carry no padding
  w.f = hi; w.f_end = lo;
  // position (r, base) on the request that holds the last position of the share
  for (;;) {
    const int N = sh.prompt_cu[w.r + 1] - sh.prompt_cu[w.r], M = sh.live_cu[w.r + 1] - sh.live_cu[w.r];
    const long long groups = walk_groups(sh, mode, M);
    const long long span = groups * (tiles_of(N, M) + pad);
    if (hi <= lo || hi - 1 < w.base + span || w.r + 1 >= sh.R) break;
    w.base += span;
    w.base_real += groups * tiles_of(N, M);
    ++w.r;
  }
}

// rel = group * T + tile; the quotient almost always fits 32 bits, where the division is an order of magnitude cheaper
__device__ __forceinline__ void split_group_tile(long long rel, int T, int& g, int& t) {
  if (rel < 0x7fffffffLL) {
    const unsigned r32 = (unsigned)rel, T32 = (unsigned)T;
    g = (int)(r32 / T32);
    t = (int)(r32 - (unsigned)g * T32);
  } else {
    g = (int)(rel / T);
    t = (int)(rel % T);
  }
}

__device__ __forceinline__ bool walker_next(Walker& w, const Shape& sh, Seg& s) {
  if (!w.reverse) {
    if (w.f >= w.f_end) return false;
    for (;;) {
      s.p0 = sh.prompt_cu[w.r]; s.N = sh.prompt_cu[w.r + 1] - s.p0;
      s.l0 = sh.live_cu[w.r]; s.M = sh.live_cu[w.r + 1] - s.l0;
      s.T = tiles_of(s.N, s.M);
      const long long span = (long long)walk_groups(sh, w.mode, s.M) * s.T;
      if (w.f < w.base + span) break;
      w.base += span;
      ++w.r;
    }
    const long long rel = w.f - w.base;
    s.r = w.r;
    split_group_tile(rel, s.T, s.g, s.t);
    s.dir = 1;
    const long long room = w.f_end - w.f;
    s.len = (int)min((long long)(s.T - s.t), room);
    s.unit_start = w.base + (long long)s.g * s.T;
    s.unit_real = s.unit_start;
    w.f += s.len;
    return true;
  }
  for (;;) {
    if (w.f <= w.f_end) return false;
    const long long last = w.f - 1;                        // highest position still to do
    for (;;) {
      s.p0 = sh.prompt_cu[w.r]; s.N = sh.prompt_cu[w.r + 1] - s.p0;
      s.l0 = sh.live_cu[w.r]; s.M = sh.live_cu[w.r + 1] - s.l0;
      s.T = tiles_of(s.N, s.M);
      if (last >= w.base) break;
      // step back to the previous request
      --w.r;
      const int N2 = sh.prompt_cu[w.r + 1] - sh.prompt_cu[w.r], M2 = sh.live_cu[w.r + 1] - sh.live_cu[w.r];
      const long long groups2 = walk_groups(sh, w.mode, M2);
      w.base -= groups2 * (tiles_of(N2, M2) + w.pad);
      w.base_real -= groups2 * tiles_of(N2, M2);
    }
    const long long rel = last - w.base;
    const int Tv = s.T + w.pad;                            // positions of a unit: padding first, then its tiles
    int tv;
    split_group_tile(rel, Tv, s.g, tv);
    const long long room = w.f - w.f_end;
    const int lenv = (int)min((long long)(tv + 1), room);
    w.f -= lenv;
    const int t_hi = tv - w.pad, t_lo = max(tv - lenv + 1 - w.pad, 0);
    if (t_hi < 0) continue;                                // this piece of the share is padding only
    s.r = w.r;
    s.t = t_hi;
    s.len = t_hi - t_lo + 1;
    s.dir = -1;
    s.unit_start = w.base + (long long)s.g * Tv;
    s.unit_real = w.base_real + (long long)s.g * s.T;
    return true;
  }
}

// CTA whose share contains flat tile f.
__host__ __device__ __forceinline__ int cta_of(long long f, long long F, int G) {
  const long long num = (f + 1) * G - 1;
  if (num < 0x7fffffffLL && F < 0x7fffffffLL) return (int)((unsigned)num / (unsigned)F);   // the usual case, a cheap division
  return (int)(num / F);
}

// =====================================================================================================
// sweep 1: per-row (max, sum of exp) over a segment of key tiles.
// part[(h*C + slot)*sumM + row] = (m2, sum of 2^(scaled logit * log2 e - m2)) with m2 an integer reference in log2 units,
// slot = 2*(cta - first cta of the row's unit) + half:
// neighbouring rows are neighbours in memory, so a warp's 32 rows of one slot are one 256-byte access.
// =====================================================================================================
template <int D>
__global__ void __launch_bounds__(kThreads, 1)
score_stats_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kp,
               const __grid_constant__ CUtensorMap map_km, Shape sh, float2* __restrict__ part, int C, long long F,
               uint32_t* __restrict__ seg_cnt, uint32_t* __restrict__ status) {
  using S = Smem<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = align_1024(smem_raw);
  const Bars bars = carve_bars(base, S::kBarOff);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + S::kMiscOff);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(base + S::kMiscOff + 4);
  if (threadIdx.x == 0) { prefetch_tmap(&map_q); prefetch_tmap(&map_kp); prefetch_tmap(&map_km); }   // kernel parameters
  block_setup(bars, 4, tmem_slot, abort_flag);
  pdl_wait();
  // Only now may sweep 2 be scheduled: once every CTA of this grid is past its wait, everything that precedes the call in
  // the stream is complete and visible, so sweep 2's loader and MMA issuer - which read nothing but the call's inputs -
  // may start before this grid has finished (its epilogue still waits for this grid's partials).
  pdl_launch_dependents();
  // sweep 2 counts finished mass partials per segment in seg_cnt; it reads them after this grid has ended
  if (blockIdx.x == 0 && seg_cnt != nullptr)
    for (int i = threadIdx.x; i < sh.R * sh.hkn; i += blockDim.x) seg_cnt[(i / sh.hkn) * sh.Hkv + sh.hk0 + i % sh.hkn] = 0u;
  const uint32_t tmem_base = *tmem_slot;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  Walker wk;
  walker_init(wk, sh, kWalkStats, false, F);
  Seg s;

  if (warp == 0) {
    if (lane == 0) {
      int kt_it = 0, q_it = 0;
      bool ok = true;
      while (ok && walker_next(wk, sh, s)) {
        const int qp_n = (s.M + kQBlock - 1) / kQBlock;
        const int h = sh.hk0 * sh.g + s.g / qp_n, q0 = (s.g % qp_n) * kQBlock, hk = h / sh.g;
        if (!(ok = mbar_wait(bars.qempty, q_it & 1, abort_flag, status, 0x100))) break;   // the MMA warp released the old block
        mbar_expect_tx(bars.qfull, S::kQBytes);
        for (int b = 0; b < S::kBoxes; ++b) tma_load_3d(base + S::kQOff + b * S::kQBoxBytes, &map_q, bars.qfull, b * 64, h, s.l0 + q0);
        ++q_it;
        for (int it = 0; it < s.len; ++it, ++kt_it) {
          const int stage = kt_it % kStages, use = kt_it / kStages;
          if (!(ok = mbar_wait(bars.empty + stage, (use & 1) ^ 1, abort_flag, status, 0x101))) break;
          const KeyTile kt = key_tile(s.t + it, s.p0, s.N, s.l0, s.M);
          mbar_expect_tx(bars.full + stage, S::kKBytes);
          for (int b = 0; b < S::kBoxes; ++b)
            tma_load_3d(base + S::kKOff + stage * S::kKBytes + b * S::kKBoxBytes, kt.prompt ? &map_kp : &map_km, bars.full + stage,
                        b * 64, hk, kt.token);
        }
      }
      if (!ok) drain_loads(bars, kt_it);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(kTile, kTile);
      const uint32_t q_lo_base = smem_desc_lo(smem_u32(base + S::kQOff));
      const uint32_t k_lo_base = smem_desc_lo(smem_u32(base + S::kKOff));
      int kt_it = 0, q_it = 0;
      uint32_t cnt[2] = {0u, 0u};                            // tiles issued per query tile
      bool ok = true;
      while (ok && walker_next(wk, sh, s)) {
        const int qp_n = (s.M + kQBlock - 1) / kQBlock;
        const int q0 = (s.g % qp_n) * kQBlock;
        const int n_qtiles = (s.M - q0 > kTile) ? 2 : 1;
        umma_commit(bars.qempty);                            // every MMA that read the resident queries has been issued
        if (!(ok = mbar_wait(bars.qfull, q_it & 1, abort_flag, status, 0x102))) break;
        ++q_it;
        tc_fence_after();
        for (int it = 0; ok && it < s.len; ++it, ++kt_it) {
          const int stage = kt_it % kStages, use = kt_it / kStages;
          if (!(ok = mbar_wait(bars.full + stage, use & 1, abort_flag, status, 0x103))) break;
          tc_fence_after();
          const uint32_t k_lo = k_lo_base + stage * (S::kKBytes >> 4);
          for (int a = 0; a < n_qtiles; ++a) {
            const int acc = a * 2 + (cnt[a] & 1);
            if (!(ok = mbar_wait(bars.tempty + acc, ((cnt[a] >> 1) & 1) ^ 1, abort_flag, status, 0x104))) break;
            tc_fence_after();
            const uint32_t q_lo = q_lo_base + ((a * kTile * 128) >> 4);
#pragma unroll
            for (int kk = 0; kk < (D / 16) * MASKKV_DBG_KSTEPS / 8; ++kk) {
              const uint32_t qo = ((kk >> 2) * S::kQBoxBytes + (kk & 3) * 32) >> 4;
              const uint32_t ko = ((kk >> 2) * S::kKBoxBytes + (kk & 3) * 32) >> 4;
              umma_ss(tmem_base + acc * kTile, make_desc(q_lo + qo, kDescHiSw128), make_desc(k_lo + ko, kDescHiSw128), idesc, kk > 0);
            }
            umma_commit(bars.tfull + acc);
            ++cnt[a];
          }
          umma_commit(bars.empty + stage);
        }
      }
    }
  } else {
    // Four warpgroups: query tile a = wg >> 1, and of each 128-key accumulator the 64-column half (wg & 1).
    // Each (row, half) keeps its own running (max, sum); the merge kernel combines the halves like any two chunks.
    const int wg = (warp - 2) >> 2;
    const int a = wg >> 1, half = wg & 1;
    const int lane_group = warp & 3;                        // TMEM lanes this warp may read
    const int row = lane_group * 32 + lane;                 // query inside the tile
    const float cs = sh.scale * kLog2e;
    uint32_t cnt = 0;
    bool ok = true;
    while (ok && walker_next(wk, sh, s)) {
      const int qp_n = (s.M + kQBlock - 1) / kQBlock;
      const int h = sh.hk0 * sh.g + s.g / qp_n, q0 = (s.g % qp_n) * kQBlock;
      const int n_qtiles = (s.M - q0 > kTile) ? 2 : 1;
      if (a >= n_qtiles) continue;
      // The row's reference m2 is an INTEGER in log2 units, at least the largest scaled logit seen so far, and
      // l = sum 2^(s * cs - m2).  An integer reference costs nothing (any reference at or above the maximum will do) and
      // lets the polynomial path fold it into its magic number; merging partials is then exact (powers of two).
      float m2 = -INFINITY, l = 0.f;
      // a chunk's maximum is a tree of 3-input max
      auto chunk_max = [&](const float* v) {
        float t[11];
#pragma unroll
        for (int c = 0; c < 10; ++c) t[c] = max3(v[3 * c], v[3 * c + 1], v[3 * c + 2]);
        t[10] = fmaxf(v[30], v[31]);
        return fmaxf(max3(max3(t[0], t[1], t[2]), max3(t[3], t[4], t[5]), max3(t[6], t[7], t[8])), fmaxf(t[9], t[10]));
      };
      auto chunk_sum = [&](const float* v, float ref2) {   // every exponential on the special-function unit
        const float neg = -ref2;
        const uint64_t cs2 = pack2(cs, cs), neg2 = pack2(neg, neg);
        uint64_t acc_a = pack2(0.f, 0.f), acc_b = pack2(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
          float x0, x1, x2, x3;
          unpack2(fma2(pack2(v[c], v[c + 1]), cs2, neg2), x0, x1);
          unpack2(fma2(pack2(v[c + 2], v[c + 3]), cs2, neg2), x2, x3);
          acc_a = add2(acc_a, pack2(ex2(x0), ex2(x1)));
          acc_b = add2(acc_b, pack2(ex2(x2), ex2(x3)));
        }
        float l0, l1;
        unpack2(add2(acc_a, acc_b), l0, l1);
        return l0 + l1;
      };
      // kStatsPolyPairs of every eight pairs as a polynomial on the FMA pipes, the others on the special-function unit;
      // the two kinds alternate so that both units have work in flight.  All 32 logits must be finite.
      auto chunk_sum_mixed = [&](const float* v, float ref2) {
        const float neg = -ref2, mk = kExpMagic - ref2;     // an integer: exact
        const uint64_t cs2 = pack2(cs, cs), neg2 = pack2(neg, neg), mk2 = pack2(mk, mk);
        uint64_t acc_a = pack2(0.f, 0.f), acc_b = pack2(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          const uint64_t v2 = pack2(v[c], v[c + 1]);
          if (poly_pair(c >> 1, kStatsPolyPairs)) {
            acc_b = add2(acc_b, exp2_poly_pair<2>(v2, cs2, mk2));
          } else {
            float x0, x1;
            unpack2(fma2(v2, cs2, neg2), x0, x1);
            acc_a = add2(acc_a, pack2(ex2(x0), ex2(x1)));
          }
        }
        float l0, l1;
        unpack2(add2(acc_a, acc_b), l0, l1);
        return l0 + l1;
      };
      auto absorb = [&](float* v, int col0, int valid) {
        const bool ragged = valid - col0 < 32;               // only the last tile of a request's prompt or mask keys
        if (ragged) {
#pragma unroll
          for (int c = 0; c < 32; ++c) if (col0 + c >= valid) v[c] = -INFINITY;
        }
        const float cm2 = chunk_max(v) * cs;
        if (cm2 > m2) { const float nm = ceilf(cm2); l *= ex2(m2 - nm); m2 = nm; }
        l += (ragged || kStatsPolyPairs == 0) ? chunk_sum(v, m2) : chunk_sum_mixed(v, m2);
      };
      // Rolling double buffer over the chunk stream (tile 0: c0, c1; tile 1: c0, c1; ...): while one 32-column chunk
      // is being exponentiated the next one - possibly of the next tile - is already on its way from tensor memory.
      const int col0 = half * 64;
      const uint32_t lane_addr = tmem_base + ((uint32_t)(lane_group * 32) << 16) + col0;
      float va[32], vb[32];
      int valid = 0;
      if (s.len > 0) {
        if ((ok = mbar_wait(bars.tfull + a * 2 + (cnt & 1), (cnt >> 1) & 1, abort_flag, status, 0x105))) {
          tc_fence_after();
          valid = key_tile(s.t, s.p0, s.N, s.l0, s.M).valid;
          tmem_ld32(lane_addr + (a * 2 + (cnt & 1)) * kTile, va);
        }
      }
      for (int it = 0; ok && it < s.len; ++it, ++cnt) {
        const int acc = a * 2 + (cnt & 1);
        // chunk 0 of this tile is in flight (into va); start chunk 1 behind it
        tmem_ld_wait();
        tmem_ld32(lane_addr + acc * kTile + 32, vb);
#ifdef MASKKV_DBG_NOMATH
        l += va[5];
#else
        if (valid > col0) absorb(va, col0, valid);
#endif
        tmem_ld_wait();
        tc_fence_before();
        mbar_arrive(bars.tempty + acc);                     // both chunks of this thread are in registers
        const int valid_now = valid;
        if (it + 1 < s.len) {                               // chunk 0 of the next tile goes out before chunk 1 is processed
          const uint32_t c2n = cnt + 1;
          if (!(ok = mbar_wait(bars.tfull + a * 2 + (c2n & 1), (c2n >> 1) & 1, abort_flag, status, 0x105))) break;
          tc_fence_after();
          valid = key_tile(s.t + it + 1, s.p0, s.N, s.l0, s.M).valid;
          tmem_ld32(lane_addr + (a * 2 + (c2n & 1)) * kTile, va);
        }
#ifdef MASKKV_DBG_NOMATH
        l += vb[7];
#else
        if (valid_now > col0 + 32) absorb(vb, col0 + 32, valid_now);
#endif
      }
      if (!ok) continue;
      const int i = q0 + a * kTile + row;
      const int slot = 2 * ((int)blockIdx.x - cta_of(s.unit_start, F, gridDim.x)) + half;
      if (i < s.M) part[((long long)h * C + slot) * sh.sumM + s.l0 + i] = make_float2(m2, l);
    }
  }
  block_teardown(tmem_base);
}

// log2 sum_j exp(s_j) of query row `row` (index over all requests) of head h: merge of the partials the CTAs of sweep 1
// left for the row's unit, which starts at flat tile `unit_start` of that sweep's walk and has T tiles.  The partials'
// references are integers in log2 units, so bringing them to a common one multiplies by exact powers of two.
// F, G: flat tile count and grid of sweep 1.
__device__ __noinline__ float merged_lse2(const float2* __restrict__ part, int C, int sumM, long long F, int G,
                                             long long unit_start, int T, int h, int row) {
  const int slots = 2 * (cta_of(unit_start + T - 1, F, G) - cta_of(unit_start, F, G) + 1);
  const float2* p = part + (long long)h * C * sumM + row;         // slot c at p[c * sumM]
  // the loads of a batch are issued together (a row has 4 to 8 partials on a long prompt)
  float m = -INFINITY, l = 0.f;
  for (int c0 = 0; c0 < slots; c0 += 8) {
    float2 v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = c0 + k < slots ? p[(long long)(c0 + k) * sumM] : make_float2(-INFINITY, 0.f);
    float bm = m;
#pragma unroll
    for (int k = 0; k < 8; ++k) bm = fmaxf(bm, v[k].x);
    if (bm == -INFINITY) continue;
    l *= ex2(m - bm);
#pragma unroll
    for (int k = 0; k < 8; ++k) l += v[k].y * ex2(v[k].x - bm);
    m = bm;
  }
  return m + __log2f(l);                                          // special-function logarithm (relative error 2^-22)
}

// One thread per (h, row): lse[h*sumM + row].  Only launched when sweep 2 does not run on the tensor-core kernel
// (which merges the partials itself).
__global__ void score_merge_stats_tc(Shape sh, const float2* __restrict__ part, int C, long long F, int G,
                                     float* __restrict__ lse) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= (long long)sh.H * sh.sumM) return;
  const int h = (int)(t / sh.sumM), row = (int)(t % sh.sumM);      // launched over all heads (hk0 = 0, hkn = H_kv)
  const int r = find_request(sh.live_cu, sh.R, row);
  long long base = 0;
  for (int r2 = 0; r2 < r; ++r2) {
    const int N2 = sh.prompt_cu[r2 + 1] - sh.prompt_cu[r2], M2 = sh.live_cu[r2 + 1] - sh.live_cu[r2];
    base += (long long)walk_groups(sh, kWalkStats, M2) * tiles_of(N2, M2);
  }
  const int N = sh.prompt_cu[r + 1] - sh.prompt_cu[r], l0 = sh.live_cu[r], M = sh.live_cu[r + 1] - l0;
  const int T = tiles_of(N, M), qp_n = (M + kQBlock - 1) / kQBlock;
  lse[t] = merged_lse2(part, C, sh.sumM, F, G, base + ((long long)h * qp_n + (row - l0) / kQBlock) * T, T, h, row) * kLn2;
}

// =====================================================================================================
// sweep 2: column sums, a thread per key.
//
// One query block (at most 256 voters) per KV head in every request (colpart == nullptr): the walk's groups are the KV
// heads, and scores[hk][p0 + j] = sum over the block's rows of w_i * exp(s_ij - lse_i) is final.  The attention masses
// are summed on the way: mass_part[(r*H_kv + hk)*Tmax*8 + slot] = (sum over prompt keys, sum over mask keys) one warp
// of one CTA saw, and the warp that completes a segment's count adds the slots into mass_p / mass_m [r*H_kv + hk].
//
// Several query blocks per KV head (grouped heads, more than 256 voters): the walk's groups are (query head, block) as
// in sweep 1, so a CTA keeps one block of queries resident over a long run of key tiles, and block b of KV head hk
// leaves its column sums in colpart[(b*H_kv + hk)*(sum_N + sum_M) + key] (mask keys behind the prompt keys);
// score_group_reduce adds the blocks up in block order and forms the masses.
// =====================================================================================================
template <int D>
__global__ void __launch_bounds__(kThreads, 1)
score_colsum_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kp,
                const __grid_constant__ CUtensorMap map_km, Shape sh, const float* __restrict__ lse,
                const float2* __restrict__ part, int C, long long F1, int G1,
                const float* __restrict__ w, float* __restrict__ scores, float* __restrict__ colpart,
                float2* __restrict__ mass_part, int Tmax, uint32_t* __restrict__ seg_cnt, float* __restrict__ mass_p,
                float* __restrict__ mass_m, long long F, float* __restrict__ scores_live, uint32_t* __restrict__ status) {
  using S = Smem<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = align_1024(smem_raw);
  const Bars bars = carve_bars(base, S::kBarOff);
  float* c2s = reinterpret_cast<float*>(base + S::kC2Off);
  float* s2s = reinterpret_cast<float*>(base + S::kS2Off);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + S::kMiscOff);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(base + S::kMiscOff + 4);
  pdl_launch_dependents();
  if (threadIdx.x == 0) { prefetch_tmap(&map_q); prefetch_tmap(&map_kp); prefetch_tmap(&map_km); }   // kernel parameters
  block_setup(bars, 2, tmem_slot, abort_flag);
  // No wait here: the loader and the MMA issuer read only the call's inputs, which are visible (sweep 1 releases this grid
  // after its own wait); the epilogue waits for sweep 1's results below.
  const uint32_t tmem_base = *tmem_slot;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool split = colpart != nullptr;
  Walker wk;
  walker_init(wk, sh, split ? kWalkColsumSplit : kWalkColsum, true, F, kColsumPad);
  Seg s;
  int last_r = -1, last_g = -1;                             // the (request, group) whose queries are resident
  // Both walks of sweep 2 number their tiles exactly like sweep 1 (KV heads = query heads x blocks when there is one
  // block per KV head; the same (query head, block) groups otherwise), so a run's unit_real is also the flat index at
  // which sweep 1 started the rows' unit: that is all the merge of its partials needs.
  // group of a run -> query head, KV head, first query of the block, index of the block among the KV head's blocks
  auto unit_of = [&](const Seg& sg, int& h, int& hk, int& q0, int& blk) {
    if (!split) { h = hk = sh.hk0 + sg.g; q0 = 0; blk = 0; return; }
    const int qp_n = (sg.M + kQBlock - 1) / kQBlock;
    h = sh.hk0 * sh.g + sg.g / qp_n; hk = h / sh.g; q0 = (sg.g % qp_n) * kQBlock; blk = (h % sh.g) * qp_n + sg.g % qp_n;
  };

  if (warp == 0) {
    if (lane == 0) {
      int kt_it = 0, q_it = 0;
      bool ok = true;
      while (ok && walker_next(wk, sh, s)) {
        int h, hk, q0, blk;
        unit_of(s, h, hk, q0, blk);
        if (s.r != last_r || s.g != last_g) {
          if (!(ok = mbar_wait(bars.qempty, q_it & 1, abort_flag, status, 0x201))) break;
          mbar_expect_tx(bars.qfull, S::kQBytes);
          for (int b = 0; b < S::kBoxes; ++b) tma_load_3d(base + S::kQOff + b * S::kQBoxBytes, &map_q, bars.qfull, b * 64, h, s.l0 + q0);
          ++q_it;
        }
        last_r = s.r; last_g = s.g;
        for (int tl = 0; tl < s.len; ++tl, ++kt_it) {
          const int stage = kt_it % kStages, use = kt_it / kStages;
          if (!(ok = mbar_wait(bars.empty + stage, (use & 1) ^ 1, abort_flag, status, 0x202))) break;
          const KeyTile kt = key_tile(s.t + s.dir * tl, s.p0, s.N, s.l0, s.M);
          mbar_expect_tx(bars.full + stage, S::kKBytes);
          for (int b = 0; b < S::kBoxes; ++b)
            tma_load_3d(base + S::kKOff + stage * S::kKBytes + b * S::kKBoxBytes, kt.prompt ? &map_kp : &map_km,
                        bars.full + stage, b * 64, hk, kt.token);
        }
      }
      if (!ok) drain_loads(bars, kt_it);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int kt_it = 0, q_it = 0, base_par = 0;
      uint32_t uses[2] = {0u, 0u};
      bool ok = true;
      const uint32_t q_lo_base = smem_desc_lo(smem_u32(base + S::kQOff));
      const uint32_t k_lo_base = smem_desc_lo(smem_u32(base + S::kKOff));
      while (ok && walker_next(wk, sh, s)) {
        int h, hk, q0, blk;
        unit_of(s, h, hk, q0, blk);
        const int n_mma = (min(kQBlock, s.M - q0) + 31) & ~31;             // columns the epilogue will read
        const uint32_t idesc = idesc_bf16_f32(kTile, n_mma);
        if (s.r != last_r || s.g != last_g) {
          umma_commit(bars.qempty);                          // every MMA that read the resident queries has been issued
          if (!(ok = mbar_wait(bars.qfull, q_it & 1, abort_flag, status, 0x203))) break;
          ++q_it;
          tc_fence_after();
        }
        last_r = s.r; last_g = s.g;
        for (int tl = 0; tl < s.len; ++tl, ++kt_it) {
          const int stage = kt_it % kStages, use = kt_it / kStages, buf = (tl + base_par) & 1;
          if (!(ok = mbar_wait(bars.full + stage, use & 1, abort_flag, status, 0x204))) break;
          if (!(ok = mbar_wait(bars.tempty + buf, (uses[buf] & 1) ^ 1, abort_flag, status, 0x205))) break;
          tc_fence_after();
          const uint32_t k_lo = k_lo_base + stage * (S::kKBytes >> 4);
#pragma unroll
          for (int kk = 0; kk < (D / 16) * MASKKV_DBG_KSTEPS / 8; ++kk) {
            const uint32_t ko = ((kk >> 2) * S::kKBoxBytes + (kk & 3) * 32) >> 4;
            const uint32_t qo = ((kk >> 2) * S::kQBoxBytes + (kk & 3) * 32) >> 4;
            umma_ss(tmem_base + buf * kQBlock, make_desc(k_lo + ko, kDescHiSw128), make_desc(q_lo_base + qo, kDescHiSw128), idesc, kk > 0);
          }
          umma_commit(bars.empty + stage);
          umma_commit(bars.tfull + buf);
          ++uses[buf];
        }
        base_par ^= s.len & 1;
      }
    }
  } else {
    // Four warpgroups: accumulator buf = wg >> 1, and of its (up to) 256 query columns the 128-column half (wg & 1).
    // The two halves of a key's sum meet in shared memory (one named barrier per tile per pair); the half-0 thread
    // owns the key from then on.  Inside a run the tile -> accumulator map is fixed, (tl + base_par) & 1; base_par
    // carries the alternation across runs.  After a failed wait a thread skips the arithmetic but still walks the
    // loops, so that every thread reaches every named barrier.
    const int wg = (warp - 2) >> 2;
    const int buf = wg >> 1, half = wg & 1;
    const int lane_group = warp & 3;
    const int row = lane_group * 32 + lane;                 // key inside the tile
    const float cs = sh.scale * kLog2e;
    const uint32_t taddr = tmem_base + ((uint32_t)(lane_group * 32) << 16) + buf * kQBlock + half * kTile;
    float* xch = reinterpret_cast<float*>(base + S::kXchOff) + buf * 2 * kTile;
    const long long keys_total = (long long)sh.sumN + sh.sumM;
    uint32_t uses = 0, c2_it = 0;
    int base_par = 0;
    bool ok = true;
    const float* c2 = c2s;
    const float* s2 = s2s;
    // Attention mass of the segment in hand (one query block per KV head only), summed over the tiles this warp
    // finished (half-0 warps).  When the walk leaves the segment the warp stores its pair in slot
    // (CTA - first CTA of the segment) * 8 + warp and counts itself in; the warp that completes the count adds the slots
    // up, always in slot order.
    int cur_seg = -1, cur_T = 0;
    long long cur_start = 0;
    float run_p = 0.f, run_m = 0.f;
    pdl_wait();                                             // sweep 1's partials (or lse), the cleared segment counters
    auto flush = [&]() {
      if (cur_seg < 0 || half != 0) return;
      const int first = cta_of(cur_start + kColsumPad, F, gridDim.x);          // the CTA with the segment's first tile
      const unsigned slots = 8u * (unsigned)(cta_of(cur_start + kColsumPad + cur_T - 1, F, gridDim.x) - first + 1);
      float2* mp = mass_part + (long long)cur_seg * Tmax * 8;
      unsigned last = 0;
      if (lane == 0) {
        mp[((int)blockIdx.x - first) * 8 + buf * 4 + lane_group] = make_float2(run_p, run_m);
        __threadfence();
        last = atomicAdd(seg_cnt + cur_seg, 1u) + 1u == slots;
      }
      if (__shfl_sync(0xffffffffu, last, 0)) {
        __threadfence();
        float sum_p = 0.f, sum_m = 0.f;
        for (unsigned t = lane; t < slots; t += 32) {
          const float2 v = __ldcg(mp + t);
          sum_p += v.x;
          sum_m += v.y;
        }
        sum_p = warp_sum(sum_p);
        sum_m = warp_sum(sum_m);
        if (lane == 0) { mass_p[cur_seg] = sum_p; mass_m[cur_seg] = sum_m; }
      }
    };
    while (walker_next(wk, sh, s)) {
      int h, hk, q0, blk;
      unit_of(s, h, hk, q0, blk);
      const bool new_q = s.r != last_r || s.g != last_g;
      last_r = s.r; last_g = s.g;
      if (!split) {
        const int seg = s.r * sh.Hkv + hk;
        if (seg != cur_seg) {
          flush();
          cur_seg = seg; cur_T = s.T; cur_start = s.unit_start;
          run_p = run_m = 0.f;
        }
      }
      const int qh0 = q0 + half * kTile;                    // first voter of this warpgroup's half of the block
      const int nq = max(0, min(kTile, s.M - qh0));
      if (new_q) {
        float* c2w = c2s + (wg * 2 + (c2_it & 1)) * kTile;
        float* s2w = s2s + (wg * 2 + (c2_it & 1)) * kTile;
        ++c2_it;
        float cst = -INFINITY;                              // 2^(x - inf) = 0: rows that do not exist never vote
        if (row < nq) {
          const int i = s.l0 + qh0 + row;
          const float lse2 = part != nullptr ? merged_lse2(part, C, sh.sumM, F1, G1, s.unit_real, s.T, h, i)
                                             : lse[(long long)h * sh.sumM + i] * kLog2e;
          cst = (w ? log2f(w[i]) : 0.f) - lse2;
        }
        // Query column `row` of this half: its weight is 2^(s*cs + cst).  A column whose exponentials go to the
        // special-function unit keeps cst; one that goes to the polynomial keeps the magic number plus the integer part of
        // cst, and 2^(fraction of cst) as a factor applied when the weight is added (rows that do not vote: factor 0).
        if (poly_pair((row & 31) >> 1, kColsumPolyPairs)) {
          const bool votes = cst > -INFINITY;
          const float ci = rintf(cst);
          s2w[row] = votes ? ex2(cst - ci) : 0.f;
          cst = votes ? kExpMagic + fmaxf(ci, -200.f) : kExpMagic - 200.f;
        }
        c2w[row] = cst;
        named_barrier(1 + wg, kTile);
        c2 = c2w;
        s2 = s2w;
      }
      const int chunks = (nq + 31) >> 5;
      auto absorb = [&](const float* v, int cb, uint64_t& acc2) {
        const float4* cc = reinterpret_cast<const float4*>(c2 + cb * 32);   // per-query constants
        const float4* ss = reinterpret_cast<const float4*>(s2 + cb * 32);
        const uint64_t cs2 = pack2(cs, cs);
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
          const float4 k4 = cc[c4];
          float4 f4 = make_float4(0.f, 0.f, 0.f, 0.f);
          if (poly_pair(2 * c4, kColsumPolyPairs) || poly_pair(2 * c4 + 1, kColsumPolyPairs)) f4 = ss[c4];
          if (poly_pair(2 * c4, kColsumPolyPairs)) {
            acc2 = fma2(exp2_poly_pair<4>(pack2(v[4 * c4], v[4 * c4 + 1]), cs2, pack2(k4.x, k4.y)), pack2(f4.x, f4.y), acc2);
          } else {
            float x0, x1;
            unpack2(fma2(pack2(v[4 * c4], v[4 * c4 + 1]), cs2, pack2(k4.x, k4.y)), x0, x1);
            acc2 = add2(acc2, pack2(ex2(x0), ex2(x1)));
          }
          if (poly_pair(2 * c4 + 1, kColsumPolyPairs)) {
            acc2 = fma2(exp2_poly_pair<4>(pack2(v[4 * c4 + 2], v[4 * c4 + 3]), cs2, pack2(k4.z, k4.w)), pack2(f4.z, f4.w), acc2);
          } else {
            float x2, x3;
            unpack2(fma2(pack2(v[4 * c4 + 2], v[4 * c4 + 3]), cs2, pack2(k4.z, k4.w)), x2, x3);
            acc2 = add2(acc2, pack2(ex2(x2), ex2(x3)));
          }
        }
      };
      float* out_row = split ? colpart + ((long long)blk * sh.Hkv + hk) * keys_total : scores + (long long)hk * sh.sumN;
      for (int tl = (buf + base_par) & 1; tl < s.len; tl += 2) {
        uint64_t acc2 = pack2(0.f, 0.f);
        if (ok) ok = mbar_wait(bars.tfull + buf, uses & 1, abort_flag, status, 0x206);
        if (ok) {
          tc_fence_after();
          // four warps per scheduler hide the load latency: no register double-buffering here
#pragma unroll 1
          for (int cb = 0; cb < chunks; ++cb) {
            float v[32];
            tmem_ld32(taddr + cb * 32, v);
            tmem_ld_wait();
#ifdef MASKKV_DBG_RELEASE_AT
            if (cb == MASKKV_DBG_RELEASE_AT) { tc_fence_before(); mbar_arrive(bars.tempty + buf); }
#else
            if (cb + 1 == chunks) { tc_fence_before(); mbar_arrive(bars.tempty + buf); }   // last logits are in registers
#endif
#ifdef MASKKV_DBG_NOMATH
            acc2 = add2(acc2, pack2(v[3], v[9]));
#else
            absorb(v, cb, acc2);
#endif
          }
          if (chunks == 0) { tc_fence_before(); mbar_arrive(bars.tempty + buf); }
        }
        float a0, a1;
        unpack2(acc2, a0, a1);
        float* slot = xch + (uses & 1) * kTile;
        ++uses;
#ifdef MASKKV_DBG_NOTAIL
        slot[row] = a0 + a1;
        continue;
#endif
        if (half == 1) slot[row] = a0 + a1;
        named_barrier(5 + buf, 2 * kTile);                  // the pair's two halves of this tile are done
        if (half == 1 || !ok) continue;
        float acc = (a0 + a1) + slot[row];
        const KeyTile kt = key_tile(s.t + s.dir * tl, s.p0, s.N, s.l0, s.M);
        if (split) {                                        // prompt keys, then mask keys, of every request
          if (row < kt.valid) out_row[(kt.prompt ? 0 : sh.sumN) + kt.token + row] = acc;
          continue;
        }
        if (row >= kt.valid) acc = 0.f;
        if (kt.prompt && row < kt.valid) out_row[kt.token + row] = acc;
        if (scores_live != nullptr && !kt.prompt && row < kt.valid) scores_live[(long long)hk * sh.sumM + kt.token + row] = acc;
        acc = warp_sum(acc);
        if (kt.prompt) run_p += acc; else run_m += acc;
      }
      base_par ^= s.len & 1;
    }
    flush();
  }
  block_teardown(tmem_base);
}

// Several query blocks per KV head: scores[hk][p0 + j] = sum over the blocks, in block order, of their column sums, and
// the tile's share of the attention masses as the FP32-pipe sweep leaves it (mass_part[((r*H_kv + hk)*Tmax + t)*4 + warp],
// summed by score_mass_reduce).  A request without voters has no blocks: zeros.  grid (Tmax, H_kv, R), 128 threads.
__global__ void score_group_reduce(Shape sh, const float* __restrict__ colpart, float* __restrict__ scores,
                                   float* __restrict__ scores_live, float2* __restrict__ mass_part, int Tmax) {
  const int t = blockIdx.x, hk = blockIdx.y, r = blockIdx.z;
  const int p0 = sh.prompt_cu[r], N = sh.prompt_cu[r + 1] - p0;
  const int l0 = sh.live_cu[r], M = sh.live_cu[r + 1] - l0;
  if (t >= tiles_of(N, M)) return;
  const KeyTile kt = key_tile(t, p0, N, l0, M);
  const int blocks = M <= 0 ? 0 : sh.g * ((M + kQBlock - 1) / kQBlock);
  const long long keys_total = (long long)sh.sumN + sh.sumM;
  const int j = threadIdx.x;
  float acc = 0.f;
  if (j < kt.valid) {
    const float* src = colpart + (long long)hk * keys_total + (kt.prompt ? 0 : sh.sumN) + kt.token + j;
    for (int b = 0; b < blocks; ++b) acc += src[(long long)b * sh.Hkv * keys_total];
    if (kt.prompt) scores[(long long)hk * sh.sumN + kt.token + j] = acc;
    else if (scores_live != nullptr) scores_live[(long long)hk * sh.sumM + kt.token + j] = acc;
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0)
    mass_part[((long long)(r * sh.Hkv + hk) * Tmax + t) * 4 + (threadIdx.x >> 5)] = kt.prompt ? make_float2(acc, 0.f) : make_float2(0.f, acc);
}

// Requests without voters (M = 0): every score is zero and so are the masses.  grid (tiles, H_kv, R).
__global__ void score_zero_fill(Shape sh, float* __restrict__ scores, float* __restrict__ mass_p, float* __restrict__ mass_m) {
  const int t = blockIdx.x, hk = blockIdx.y, r = blockIdx.z;
  const int p0 = sh.prompt_cu[r], N = sh.prompt_cu[r + 1] - p0;
  const int M = sh.live_cu[r + 1] - sh.live_cu[r];
  if (M > 0) return;
  if (t == 0 && threadIdx.x == 0) { mass_p[r * sh.Hkv + hk] = 0.f; mass_m[r * sh.Hkv + hk] = 0.f; }
  if (t * kTile >= N) return;
  const int j = t * kTile + threadIdx.x;
  if (j < N) scores[(long long)hk * sh.sumN + p0 + j] = 0.f;
}

// =====================================================================================================
// host side
// =====================================================================================================
namespace {

struct Maps { CUtensorMap q, kp, km; };

bool build_maps(maskkv_ctx* ctx, const Shape& sh, const void* q, const void* kp, const void* km, Maps* m) {
  // a tensor without rows still needs a valid map: point it at the query tensor (it is never dereferenced)
  const void* kp_base = sh.sumN > 0 ? kp : q;
  const uint64_t kp_rows = sh.sumN > 0 ? (uint64_t)sh.sumN : 1;
  return make_tmap_rows(ctx->encode_tiled, &m->q, q, sh.d, sh.H, sh.sumM, sh.q_hs * 2, sh.q_ts * 2, kQBlock) &&
         make_tmap_rows(ctx->encode_tiled, &m->kp, kp_base, sh.d, sh.Hkv, kp_rows, sh.kv_hs * 2, sh.kv_ts * 2, kTile) &&
         make_tmap_rows(ctx->encode_tiled, &m->km, km, sh.d, sh.Hkv, sh.sumM, sh.kv_hs * 2, sh.kv_ts * 2, kTile);
}

// F of the walk: tiles over all (request, group) pairs, from the host's copy of the lengths.
long long flat_tiles(const Shape& sh, const int32_t* prompt_cu, const int32_t* live_cu, int mode) {
  const int pad = mode == kWalkStats ? 0 : kColsumPad;
  long long F = 0;
  for (int r = 0; r < sh.R; ++r) {
    const int N = prompt_cu[r + 1] - prompt_cu[r], M = live_cu[r + 1] - live_cu[r];
    F += (long long)walk_groups(sh, mode, M) * ((N + kTile - 1) / kTile + (M + kTile - 1) / kTile + pad);
  }
  return F;
}

// The opt-in shared-memory size is an attribute of the kernel on ONE device: remembered per device, set with that device
// current (the entry points hold a device guard).
template <int D>
cudaError_t set_smem_attr(int device) {
  static bool done[kMaxAttrDevices] = {};
  if (device < 0 || device >= kMaxAttrDevices) return cudaErrorInvalidDevice;
  if (done[device]) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(score_stats_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::kDynamic);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(score_colsum_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::kDynamic);
  done[device] = e == cudaSuccess;
  return e;
}

}  // namespace

int score_tc_max_chunks(const maskkv_ctx* ctx, const Shape& sh) {
  // partials per row in sweep 1: two per CTA that touches the row's unit.  A unit of T tiles lies inside a request
  // that contributes at least H*T tiles to the walk, so a CTA's share is at least floor(H*T/G) >= H*T/(2G) tiles (or
  // one tile) and the unit spans at most 2*ceil(G/H) + 1 shares - and never more than T.
  const int T = (sh.maxN + kTile - 1) / kTile + (sh.maxM + kTile - 1) / kTile;
  const int heads = sh.hkn * sh.g;                         // query heads one launch walks
  const int span = 2 * ((ctx->sm_count + heads - 1) / heads) + 2;
  return 2 * (span < T ? span : T);
}

int score_tc_max_tiles(const Shape& sh) { return (sh.maxN + kTile - 1) / kTile + (sh.maxM + kTile - 1) / kTile; }

bool score_tc_supported(const maskkv_ctx* ctx, const Shape& sh) {
  return sh.dtype == MASKKV_BF16 && ctx->encode_tiled != nullptr && sh.sumM > 0 &&
         ctx->smem_optin >= Smem<128>::kDynamic;
}

int launch_score_stats_tc(maskkv_ctx* ctx, const Shape& sh, const int32_t* prompt_cu_host, const int32_t* live_cu_host,
                          const void* q, const void* kp, const void* km, float2* part, int C, uint32_t* seg_cnt, cudaStream_t st) {
  Maps m;
  if (!build_maps(ctx, sh, q, kp, km, &m)) return 1;
  const long long F = flat_tiles(sh, prompt_cu_host, live_cu_host, kWalkStats);
  if (F <= 0) return 1;
  const int grid = (int)(F < ctx->sm_count ? F : ctx->sm_count);
  cudaError_t le;
  if (sh.d == 128) {
    if (set_smem_attr<128>(ctx->device) != cudaSuccess) return 1;
    le = launch_overlapped(score_stats_tc<128>, dim3(grid), dim3(kThreads), Smem<128>::kDynamic, st, m.q, m.kp, m.km, sh, part, C, F, seg_cnt,
                      ctx->status_dev);
  } else {
    if (set_smem_attr<64>(ctx->device) != cudaSuccess) return 1;
    le = launch_overlapped(score_stats_tc<64>, dim3(grid), dim3(kThreads), Smem<64>::kDynamic, st, m.q, m.kp, m.km, sh, part, C, F, seg_cnt,
                      ctx->status_dev);
  }
  if (le != cudaSuccess) { cudaGetLastError(); return 1; }   // a refused launch: the caller falls back and flags it
  return 0;
}

void launch_score_merge_tc(maskkv_ctx* ctx, const Shape& sh, const int32_t* prompt_cu_host, const int32_t* live_cu_host,
                           const float2* part, int C, float* lse, cudaStream_t st) {
  const long long F = flat_tiles(sh, prompt_cu_host, live_cu_host, kWalkStats);
  const int grid = (int)(F < ctx->sm_count ? F : ctx->sm_count);
  const long long rows = (long long)sh.H * sh.sumM;
  score_merge_stats_tc<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(sh, part, C, F, grid, lse);
}

bool score_tc_split_blocks(const Shape& sh) { return sh.g > 1 || sh.maxM > kQBlock; }

size_t score_tc_colpart_bytes(const Shape& sh) {
  if (!score_tc_split_blocks(sh)) return 0;
  const size_t blocks = (size_t)sh.g * (size_t)((sh.maxM + kQBlock - 1) / kQBlock);
  return sizeof(float) * blocks * (size_t)sh.Hkv * ((size_t)sh.sumN + (size_t)sh.sumM);
}

int launch_score_colsum_tc(maskkv_ctx* ctx, const Shape& sh, const int32_t* prompt_cu_host, const int32_t* live_cu_host,
                           const void* q, const void* kp, const void* km, const float* lse, const float2* part, int C,
                           const float* w, float* scores, float* colpart, float2* mass_part, int Tmax, uint32_t* seg_cnt,
                           float* mass_p, float* mass_m, float* scores_live, bool any_without_voters, cudaStream_t st, int* launches) {
  Maps m;
  if (!build_maps(ctx, sh, q, kp, km, &m)) return 1;
  const bool split = score_tc_split_blocks(sh);
  if (split && colpart == nullptr) return 1;
  const long long F = flat_tiles(sh, prompt_cu_host, live_cu_host, split ? kWalkColsumSplit : kWalkColsum);
  if (F <= 0) return 1;
  const int grid = (int)(F < ctx->sm_count ? F : ctx->sm_count);
  const long long F1 = flat_tiles(sh, prompt_cu_host, live_cu_host, kWalkStats);   // sweep 1's walk, for its partials
  const int G1 = (int)(F1 < ctx->sm_count ? F1 : ctx->sm_count);
  if (sh.d == 128 ? set_smem_attr<128>(ctx->device) != cudaSuccess : set_smem_attr<64>(ctx->device) != cudaSuccess) return 1;
  *launches = 0;
  if (any_without_voters && !split) {                      // with several query blocks the reduce kernel writes the zeros
    dim3 gz(score_tc_max_tiles(sh), sh.Hkv, sh.R);
    score_zero_fill<<<gz, kTile, 0, st>>>(sh, scores, mass_p, mass_m);
    ++*launches;
  }
  float* cp = split ? colpart : nullptr;
  cudaError_t le;
  if (sh.d == 128)
    le = launch_overlapped(score_colsum_tc<128>, dim3(grid), dim3(kThreads), Smem<128>::kDynamic, st, m.q, m.kp, m.km, sh, lse, part, C, F1, G1,
                      w, scores, cp, mass_part, Tmax, seg_cnt, mass_p, mass_m, F, scores_live, ctx->status_dev);
  else
    le = launch_overlapped(score_colsum_tc<64>, dim3(grid), dim3(kThreads), Smem<64>::kDynamic, st, m.q, m.kp, m.km, sh, lse, part, C, F1, G1,
                      w, scores, cp, mass_part, Tmax, seg_cnt, mass_p, mass_m, F, scores_live, ctx->status_dev);
  if (le != cudaSuccess) { cudaGetLastError(); return 1; }   // a refused launch: the caller falls back and flags it
  ++*launches;
  if (split) {
    dim3 gr(Tmax, sh.Hkv, sh.R);
    score_group_reduce<<<gr, kTile, 0, st>>>(sh, colpart, scores, scores_live, mass_part, Tmax);
    ++*launches;
  }
  return 0;
}

}  // namespace tc
}  // namespace mkv

// Mask-voting scores (Eq. 6-7, sums of Eq. 14) for bf16 inputs on the 5th-generation tensor cores.
//
// The logits S = Q K^T are produced tile by tile by tcgen05.mma into tensor memory and consumed there:
// the M x (N+M) weight matrix never exists in shared or global memory.  Column sums need each row's
// final normaliser, so the product is formed twice:
//
//   sweep 1  score_stats_tc   queries on the TMEM lanes (A = 128-query tile, B = 128-key tile): the thread
//                             that owns a lane owns a softmax row and keeps its running (max, sum of exp).
//                             A CTA covers 256 queries (two accumulators) x one chunk of key tiles and
//                             writes one partial per row; a tiny kernel merges the partials into lse_i.
//   sweep 2  score_colsum_tc  keys on the TMEM lanes (A = 128-key tile, B = up to 256 queries): the owning
//                             thread reads its key's logits against every query, forms
//                             A_ij = 2^(s_ij*c - lse2_i) and sums over i in a register - the column sum
//                             needs no cross-thread reduction.
//
// Both kernels are warp-specialised: warp 0 issues TMA loads (4-stage ring of key tiles), warp 1 issues
// the MMAs, warps 2-9 are two epilogue warpgroups working on alternate accumulators so that the tensor
// pipe and the exponentials overlap.  Tensor memory: 512 columns = 2 x 256 (sweep 2) or 4 x 128 (sweep 1).
#include "score_tc.h"

#include "tc_common.cuh"

namespace mkv {
namespace tc {

constexpr int kThreads = 320;          // 10 warps: TMA, MMA, 2 x 4 epilogue
constexpr int kStages = 4;
constexpr int kTile = 128;             // keys per tile (both sweeps), queries per accumulator (sweep 1)
constexpr int kQBlock = 256;           // queries resident per CTA
constexpr int kColsumMaxTiles = 16;    // key tiles per CTA in sweep 2 (bounded by the shared-memory accumulators)
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct Smem {
  static constexpr int kBoxes = D / 64;
  static constexpr int kQBoxBytes = kQBlock * 128;          // one 64-column box of the 256 resident queries
  static constexpr int kQBytes = kBoxes * kQBoxBytes;
  static constexpr int kKBoxBytes = kTile * 128;
  static constexpr int kKBytes = kBoxes * kKBoxBytes;
  static constexpr int kQOff = 0;
  static constexpr int kKOff = kQBytes;
  static constexpr int kAccOff = kKOff + kStages * kKBytes;               // float [kColsumMaxTiles][128]
  static constexpr int kC2Off = kAccOff + kColsumMaxTiles * kTile * 4;     // float [2][256]
  static constexpr int kRedOff = kC2Off + 2 * kQBlock * 4;                 // float [8]
  static constexpr int kBarOff = kRedOff + 64;                             // mbarriers
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

// =====================================================================================================
// sweep 1: per-row (max, sum of exp) over one chunk of key tiles.
// grid (chunks, H, R * q_pairs); part[(h*sumM + row)*C + chunk] = (max of scaled logits, sum of exp).
// =====================================================================================================
template <int D>
__global__ void __launch_bounds__(kThreads, 1)
score_stats_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kp,
               const __grid_constant__ CUtensorMap map_km, Shape sh, float2* __restrict__ part, int C, int chunk_tiles,
               uint32_t* __restrict__ status) {
  using S = Smem<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = align_1024(smem_raw);
  const Bars bars = carve_bars(base, S::kBarOff);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + S::kMiscOff);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(base + S::kMiscOff + 4);

  const int q_pairs = (sh.maxM + kQBlock - 1) / kQBlock;
  const int chunk = blockIdx.x, h = blockIdx.y, r = blockIdx.z / q_pairs, qp = blockIdx.z % q_pairs;
  const int hk = h / sh.g;
  const int p0 = sh.prompt_cu[r], N = sh.prompt_cu[r + 1] - p0;
  const int l0 = sh.live_cu[r], M = sh.live_cu[r + 1] - l0;
  const int T = (N + kTile - 1) / kTile + (M + kTile - 1) / kTile;
  const int q0 = qp * kQBlock;
  const int t_begin = chunk * chunk_tiles, t_end = min(t_begin + chunk_tiles, T);
  if (q0 >= M || t_begin >= t_end) return;                 // nothing to do (uniform for the block)
  const int n_qtiles = (M - q0 > kTile) ? 2 : 1;
  const int nt = t_end - t_begin;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(bars.full + s, 1); mbar_init(bars.empty + s, 1); }
    mbar_init(bars.qfull, 1); mbar_init(bars.qempty, 1);
    for (int b = 0; b < 4; ++b) { mbar_init(bars.tfull + b, 1); mbar_init(bars.tempty + b, kTile); }
    *abort_flag = 0u;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&map_q); prefetch_tmap(&map_kp); prefetch_tmap(&map_km);
      mbar_expect_tx(bars.qfull, S::kQBytes);
      for (int b = 0; b < S::kBoxes; ++b) tma_load_3d(base + S::kQOff + b * S::kQBoxBytes, &map_q, bars.qfull, b * 64, h, l0 + q0);
      int it = 0;
      for (; it < nt; ++it) {
        const int stage = it % kStages, use = it / kStages;
        if (!mbar_wait(bars.empty + stage, (use & 1) ^ 1, abort_flag, status, 0x101)) break;
        const KeyTile kt = key_tile(t_begin + it, p0, N, l0, M);
        mbar_expect_tx(bars.full + stage, S::kKBytes);
        for (int b = 0; b < S::kBoxes; ++b)
          tma_load_3d(base + S::kKOff + stage * S::kKBytes + b * S::kKBoxBytes, kt.prompt ? &map_kp : &map_km, bars.full + stage,
                      b * 64, hk, kt.token);
      }
      if (it < nt) drain_loads(bars, it);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(kTile, kTile);
      bool ok = mbar_wait(bars.qfull, 0, abort_flag, status, 0x102);
      tc_fence_after();
      for (int it = 0; ok && it < nt; ++it) {
        const int stage = it % kStages, use = it / kStages, buf = it & 1;
        if (!(ok = mbar_wait(bars.full + stage, use & 1, abort_flag, status, 0x103))) break;
        tc_fence_after();
        const uint32_t k_addr = smem_u32(base + S::kKOff + stage * S::kKBytes);
        for (int a = 0; a < n_qtiles; ++a) {
          const int acc = a * 2 + buf;
          if (!(ok = mbar_wait(bars.tempty + acc, ((it >> 1) & 1) ^ 1, abort_flag, status, 0x104))) break;
          tc_fence_after();
          const uint32_t q_addr = smem_u32(base + S::kQOff) + a * kTile * 128;
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t adesc = smem_desc_sw128(q_addr + (kk >> 2) * S::kQBoxBytes + (kk & 3) * 32);
            const uint64_t bdesc = smem_desc_sw128(k_addr + (kk >> 2) * S::kKBoxBytes + (kk & 3) * 32);
            umma_ss(tmem_base + acc * kTile, adesc, bdesc, idesc, kk > 0);
          }
          umma_commit(bars.tfull + acc);
        }
        umma_commit(bars.empty + stage);
      }
    }
  } else {
    const int wg = (warp - 2) >> 2;                         // warpgroup = query tile
    const int lane_group = warp & 3;                        // TMEM lanes this warp may read
    const int row = lane_group * 32 + lane;                 // query inside the tile
    if (wg < n_qtiles) {
      const float cs = sh.scale * kLog2e;
      float m = -INFINITY, l = 0.f;                         // m in raw (unscaled) logits
      bool ok = true;
      for (int it = 0; ok && it < nt; ++it) {
        const int buf = it & 1, acc = wg * 2 + buf;
        if (!(ok = mbar_wait(bars.tfull + acc, (it >> 1) & 1, abort_flag, status, 0x105))) break;
        tc_fence_after();
        const int valid = key_tile(t_begin + it, p0, N, l0, M).valid;
        const uint32_t taddr = tmem_base + ((uint32_t)(lane_group * 32) << 16) + acc * kTile;
#pragma unroll 1
        for (int cb = 0; cb < kTile / 32; ++cb) {
          if (cb * 32 >= valid) break;
          float v[32];
          tmem_ld32(taddr + cb * 32, v);
          tmem_ld_wait();
          if (valid - cb * 32 < 32) {
#pragma unroll
            for (int c = 0; c < 32; ++c) if (cb * 32 + c >= valid) v[c] = -INFINITY;
          }
          float cmax = v[0];
#pragma unroll
          for (int c = 1; c < 32; ++c) cmax = fmaxf(cmax, v[c]);
          if (cmax > m) { l *= ex2((m - cmax) * cs); m = cmax; }
          const float neg = -m * cs;
#pragma unroll
          for (int c = 0; c < 32; ++c) l += ex2(fmaf(v[c], cs, neg));
        }
        tc_fence_before();
        mbar_arrive(bars.tempty + acc);
      }
      const int i = q0 + wg * kTile + row;
      if (ok && i < M) part[((long long)h * sh.sumM + l0 + i) * C + chunk] = make_float2(m * sh.scale, l);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

// =====================================================================================================
// sweep 2: column sums.  grid (tile groups, H_kv, R).
// scores[hk][p0 + j] = sum over the group's query heads and mask rows of w_i * exp(s_ij - lse_i);
// mass_part[(r*H_kv + hk)*Tmax + t] = (sum over the tile's prompt keys, sum over its mask keys).
// =====================================================================================================
template <int D>
__global__ void __launch_bounds__(kThreads, 1)
score_colsum_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kp,
                const __grid_constant__ CUtensorMap map_km, Shape sh, const float* __restrict__ lse,
                const float* __restrict__ w, float* __restrict__ scores, float2* __restrict__ mass_part, int Tmax,
                int tiles_per_cta, uint32_t* __restrict__ status) {
  using S = Smem<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = align_1024(smem_raw);
  const Bars bars = carve_bars(base, S::kBarOff);
  float* accs = reinterpret_cast<float*>(base + S::kAccOff);
  float* c2s = reinterpret_cast<float*>(base + S::kC2Off);
  float* red = reinterpret_cast<float*>(base + S::kRedOff);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + S::kMiscOff);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(base + S::kMiscOff + 4);

  const int r = blockIdx.z, hk = blockIdx.y;
  const int p0 = sh.prompt_cu[r], N = sh.prompt_cu[r + 1] - p0;
  const int l0 = sh.live_cu[r], M = sh.live_cu[r + 1] - l0;
  const int T = (N + kTile - 1) / kTile + (M + kTile - 1) / kTile;
  const int t_begin = blockIdx.x * tiles_per_cta, t_end = min(t_begin + tiles_per_cta, T);
  float2* mp = mass_part + (long long)(r * sh.Hkv + hk) * Tmax;
  // tiles of this CTA's nominal range that the request does not have: their partials must read as zero
  for (int t = max(t_begin, T) + (int)threadIdx.x; t < min(t_begin + tiles_per_cta, Tmax); t += kThreads) mp[t] = make_float2(0.f, 0.f);
  if (t_begin >= t_end) return;
  const int nt = t_end - t_begin;
  if (M == 0) {                                             // no voters: every score of the range is zero
    for (int e = threadIdx.x; e < nt * kTile; e += kThreads) {
      const int j = t_begin * kTile + e;
      if (j < N) scores[(long long)hk * sh.sumN + p0 + j] = 0.f;
    }
    for (int t = t_begin + (int)threadIdx.x; t < t_end; t += kThreads) mp[t] = make_float2(0.f, 0.f);
    return;
  }
  const int q_per_head = (M + kQBlock - 1) / kQBlock;
  const int nqb = sh.g * q_per_head;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(bars.full + s, 1); mbar_init(bars.empty + s, 1); }
    mbar_init(bars.qfull, 1); mbar_init(bars.qempty, 1);
    for (int b = 0; b < 2; ++b) { mbar_init(bars.tfull + b, 1); mbar_init(bars.tempty + b, kTile); }
    *abort_flag = 0u;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&map_q); prefetch_tmap(&map_kp); prefetch_tmap(&map_km);
      int it = 0;
      bool ok = true;
      for (int qb = 0; ok && qb < nqb; ++qb) {
        const int h = hk * sh.g + qb / q_per_head, q0 = (qb % q_per_head) * kQBlock;
        if (!(ok = mbar_wait(bars.qempty, (qb & 1) ^ 1, abort_flag, status, 0x201))) break;
        mbar_expect_tx(bars.qfull, S::kQBytes);
        for (int b = 0; b < S::kBoxes; ++b) tma_load_3d(base + S::kQOff + b * S::kQBoxBytes, &map_q, bars.qfull, b * 64, h, l0 + q0);
        for (int tl = 0; tl < nt; ++tl, ++it) {
          const int stage = it % kStages, use = it / kStages;
          if (!(ok = mbar_wait(bars.empty + stage, (use & 1) ^ 1, abort_flag, status, 0x202))) break;
          const KeyTile kt = key_tile(t_begin + tl, p0, N, l0, M);
          mbar_expect_tx(bars.full + stage, S::kKBytes);
          for (int b = 0; b < S::kBoxes; ++b)
            tma_load_3d(base + S::kKOff + stage * S::kKBytes + b * S::kKBoxBytes, kt.prompt ? &map_kp : &map_km,
                        bars.full + stage, b * 64, hk, kt.token);
        }
      }
      if (!ok) drain_loads(bars, it);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int it = 0;
      uint32_t uses[2] = {0u, 0u};
      bool ok = true;
      const uint32_t q_addr = smem_u32(base + S::kQOff);
      for (int qb = 0; ok && qb < nqb; ++qb) {
        const int q0 = (qb % q_per_head) * kQBlock;
        const int n_mma = (min(kQBlock, M - q0) + 31) & ~31;           // columns the epilogue will read
        const uint32_t idesc = idesc_bf16_f32(kTile, n_mma);
        if (!(ok = mbar_wait(bars.qfull, qb & 1, abort_flag, status, 0x203))) break;
        tc_fence_after();
        for (int tl = 0; tl < nt; ++tl, ++it) {
          const int stage = it % kStages, use = it / kStages, buf = tl & 1;
          if (!(ok = mbar_wait(bars.full + stage, use & 1, abort_flag, status, 0x204))) break;
          if (!(ok = mbar_wait(bars.tempty + buf, (uses[buf] & 1) ^ 1, abort_flag, status, 0x205))) break;
          tc_fence_after();
          const uint32_t k_addr = smem_u32(base + S::kKOff + stage * S::kKBytes);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t adesc = smem_desc_sw128(k_addr + (kk >> 2) * S::kKBoxBytes + (kk & 3) * 32);
            const uint64_t bdesc = smem_desc_sw128(q_addr + (kk >> 2) * S::kQBoxBytes + (kk & 3) * 32);
            umma_ss(tmem_base + buf * kQBlock, adesc, bdesc, idesc, kk > 0);
          }
          umma_commit(bars.empty + stage);
          umma_commit(bars.tfull + buf);
          ++uses[buf];
        }
        umma_commit(bars.qempty);
      }
    }
  } else {
    const int wg = (warp - 2) >> 2;                         // warpgroup = accumulator = parity of the local tile index
    const int lane_group = warp & 3;
    const int row = lane_group * 32 + lane;                 // key inside the tile
    const int tid_wg = ((warp - 2) & 3) * 32 + lane;
    float* c2 = c2s + wg * kQBlock;
    const float cs = sh.scale * kLog2e;
    uint32_t uses = 0;
    bool ok = true;
    // After a failed wait a thread skips the work but still walks the loops, so that every thread of the
    // warpgroup reaches every named barrier.
    for (int qb = 0; qb < nqb; ++qb) {
      const int h = hk * sh.g + qb / q_per_head, q0 = (qb % q_per_head) * kQBlock;
      const int nq = min(kQBlock, M - q0);
      named_barrier(1 + wg, kTile);                         // the previous block's constants are no longer read
      for (int e = tid_wg; e < kQBlock; e += kTile) {
        const int q = q0 + e;
        float c = INFINITY;                                 // 2^(x - inf) = 0: rows that do not exist never vote
        if (e < nq) c = lse[(long long)h * sh.sumM + l0 + q] * kLog2e - (w ? log2f(w[l0 + q]) : 0.f);
        c2[e] = c;
      }
      named_barrier(1 + wg, kTile);
      const int chunks = (nq + 31) >> 5;
      for (int tl = wg; ok && tl < nt; tl += 2) {
        if (!(ok = mbar_wait(bars.tfull + wg, uses & 1, abort_flag, status, 0x206))) break;
        ++uses;
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(lane_group * 32) << 16) + wg * kQBlock;
        float a0 = 0.f, a1 = 0.f;
#pragma unroll 1
        for (int cb = 0; cb < chunks; ++cb) {
          float v[32];
          tmem_ld32(taddr + cb * 32, v);
          tmem_ld_wait();
          const float4* cc = reinterpret_cast<const float4*>(c2 + cb * 32);
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4) {
            const float4 k4 = cc[c4];
            a0 += ex2(fmaf(v[4 * c4], cs, -k4.x));
            a1 += ex2(fmaf(v[4 * c4 + 1], cs, -k4.y));
            a0 += ex2(fmaf(v[4 * c4 + 2], cs, -k4.z));
            a1 += ex2(fmaf(v[4 * c4 + 3], cs, -k4.w));
          }
        }
        tc_fence_before();
        mbar_arrive(bars.tempty + wg);
        const float acc = a0 + a1;
        if (qb == 0) accs[tl * kTile + row] = acc; else accs[tl * kTile + row] += acc;
      }
    }
    named_barrier(3, 2 * kTile);                            // both warpgroups: all column sums are in shared memory
    if (wg == 0 && !*abort_flag) {
      for (int tl = 0; tl < nt; ++tl) {
        const KeyTile kt = key_tile(t_begin + tl, p0, N, l0, M);
        float v = accs[tl * kTile + tid_wg];
        if (tid_wg >= kt.valid) v = 0.f;
        if (kt.prompt && tid_wg < kt.valid) scores[(long long)hk * sh.sumN + kt.token + tid_wg] = v;
        v = warp_sum(v);
        if (lane == 0) red[(warp - 2) & 3] = v;
        named_barrier(1, kTile);
        if (tid_wg == 0) {
          const float s = (red[0] + red[1]) + (red[2] + red[3]);
          mp[t_begin + tl] = kt.prompt ? make_float2(s, 0.f) : make_float2(0.f, s);
        }
        named_barrier(1, kTile);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
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

// Tiles per CTA such that the grid is close to a whole number of waves over the SMs.
int pick_tiles(int tiles, long long units, int sm_count, int lo, int hi) {
  int best = lo;
  double best_eff = -1.0;
  for (int tp = lo; tp <= hi; ++tp) {
    const long long ctas = units * ((tiles + tp - 1) / tp);
    const long long waves = (ctas + sm_count - 1) / sm_count;
    // work is counted in tiles: the slowest SM processes `waves` CTAs of up to tp tiles (+1 for the query load)
    const double eff = (double)units * tiles / ((double)waves * sm_count * (tp + 1.0));
    if (eff > best_eff) { best_eff = eff; best = tp; }
  }
  return best;
}

template <int D>
cudaError_t set_smem_attr() {
  static bool done = false;
  if (done) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(score_stats_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::kDynamic);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(score_colsum_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::kDynamic);
  done = e == cudaSuccess;
  return e;
}

}  // namespace

int score_tc_max_chunks(const Shape& sh) {
  const int T = (sh.maxN + kTile - 1) / kTile + (sh.maxM + kTile - 1) / kTile;
  return (T + 3) / 4;                                       // a chunk never has fewer than 4 tiles
}

int score_tc_max_tiles(const Shape& sh) { return (sh.maxN + kTile - 1) / kTile + (sh.maxM + kTile - 1) / kTile; }

bool score_tc_supported(const maskkv_ctx* ctx, const Shape& sh) {
  return sh.dtype == MASKKV_BF16 && ctx->encode_tiled != nullptr && sh.sumM > 0 &&
         ctx->smem_optin >= Smem<128>::kDynamic;
}

int launch_score_stats_tc(maskkv_ctx* ctx, const Shape& sh, const void* q, const void* kp, const void* km, float2* part,
                          int C, int* chunk_tiles_out, cudaStream_t st) {
  Maps m;
  if (!build_maps(ctx, sh, q, kp, km, &m)) return 1;
  const int T = score_tc_max_tiles(sh);
  const int q_pairs = (sh.maxM + kQBlock - 1) / kQBlock;
  int ct = pick_tiles(T, (long long)sh.H * sh.R * q_pairs, ctx->sm_count, 4, 32);
  while ((T + ct - 1) / ct > C) ++ct;
  *chunk_tiles_out = ct;
  dim3 grid((T + ct - 1) / ct, sh.H, sh.R * q_pairs);
  if (sh.d == 128) {
    if (set_smem_attr<128>() != cudaSuccess) return 1;
    score_stats_tc<128><<<grid, kThreads, Smem<128>::kDynamic, st>>>(m.q, m.kp, m.km, sh, part, C, ct, ctx->status_dev);
  } else {
    if (set_smem_attr<64>() != cudaSuccess) return 1;
    score_stats_tc<64><<<grid, kThreads, Smem<64>::kDynamic, st>>>(m.q, m.kp, m.km, sh, part, C, ct, ctx->status_dev);
  }
  return 0;
}

int launch_score_colsum_tc(maskkv_ctx* ctx, const Shape& sh, const void* q, const void* kp, const void* km, const float* lse,
                           const float* w, float* scores, float2* mass_part, int Tmax, cudaStream_t st) {
  Maps m;
  if (!build_maps(ctx, sh, q, kp, km, &m)) return 1;
  const int T = score_tc_max_tiles(sh);
  const int tp = pick_tiles(T, (long long)sh.Hkv * sh.R, ctx->sm_count, 4, kColsumMaxTiles);
  dim3 grid((T + tp - 1) / tp, sh.Hkv, sh.R);
  if (sh.d == 128) {
    if (set_smem_attr<128>() != cudaSuccess) return 1;
    score_colsum_tc<128><<<grid, kThreads, Smem<128>::kDynamic, st>>>(m.q, m.kp, m.km, sh, lse, w, scores, mass_part, Tmax, tp,
                                                                      ctx->status_dev);
  } else {
    if (set_smem_attr<64>() != cudaSuccess) return 1;
    score_colsum_tc<64><<<grid, kThreads, Smem<64>::kDynamic, st>>>(m.q, m.kp, m.km, sh, lse, w, scores, mass_part, Tmax, tp,
                                                                     ctx->status_dev);
  }
  return 0;
}

}  // namespace tc
}  // namespace mkv

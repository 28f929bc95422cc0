// Attention of a later denoising step over [compacted prompt segment ; live keys] for bf16 inputs on
// the 5th-generation tensor cores (appendix, proof step 3: out_m = sum_j softmax(q_m k_j / sqrt(d_k)) V_j).
//
// One CTA per (128-query tile, query head, request).  Key tiles of 128 rows are walked first over the
// head's ragged segment of the compacted cache (rows [offsets[s], offsets[s+1]) of kc / vc), then over
// the request's live rows.  Per tile:
//     S = Q K^T            tcgen05.mma, operands in shared memory (TMA, 128-byte swizzle), S in tensor memory
//     P = 2^(S*c - m*c)    two threads per query row, 64 key columns each, each with an online softmax of its own
//                          (reference m, sum l) in fp32; P rounded to bf16 and written back over S
//     O_w += P_w V_w       tcgen05.mma with P read from tensor memory and V (row-major, i.e. N-major) from shared
//                          memory, accumulated over all tiles in the warpgroup's own 128 columns of tensor memory
// S/P is double-buffered so the next tile's Q K^T overlaps the softmax; Q K^T and the two P V streams are issued by
// three different threads; key and value tiles come through separate TMA rings (3 and 2 stages) and tiles beyond
// the rings are requested into L2 ahead of time.  A reference only moves when a logit exceeds it by more than 2^8
// (then the thread rescales its row of O_w in tensor memory), so nothing per tile waits for a P V product or for the
// other warpgroup; the two partial softmaxes are merged once, after the last tile, straight from tensor memory (a
// thread can read its row of both accumulators).  Columns of a ragged tile's tail
// are masked to -inf, and the matching V rows are zeroed in shared memory so that stale cache rows can never leak a
// NaN into the product.  The output tile leaves through shared memory as whole rows.
//
// The kernel is a latency chain (3-8 dependent tiles per CTA), not a throughput kernel.  Cycle stamps of one CTA:
// 2.6k cycles until the tile loop starts (set-up, wait for the previous kernel, segment offsets), 2.3k more until the
// first S is ready (tensor maps, Q and K from L2, first MMA group), then about 2.0k per tile - 0.3k reading S and
// finding the row maximum, 1.4k for the 128 x 128 exponentials (1,024 cycles of the special-function unit by
// themselves; the two warpgroups stay in phase because the S buffers are shared), packing and the store of P - and
// 2.5k to merge, normalise and store.  When units are few and their key segments long, a cluster of two CTAs shares a
// unit: each walks half of the tiles and CTA 1 hands its (max, sum, output) to CTA 0 through distributed shared
// memory; that merge costs about three tiles' time, so it is used from eight tiles per unit on.
#include "attend_tc.h"

#include <cooperative_groups.h>

#include "tc_common.cuh"

namespace mkv {
namespace tc {

// warp 0: TMA; warp 1: issues Q K^T; warps 2-9: two softmax warpgroups (thread = one query row, 64 key columns of every
// tile); warps 10, 11: issue P V of warpgroup 0 / 1.
template <int D> struct AWgs { static constexpr int kNW = 2; static constexpr int kThreads = 64 + 128 * kNW + 32 * kNW; static constexpr int kPvWarp = 2 + 4 * kNW; };
constexpr int kATile = 128;
constexpr int kAKStages = 3;            // key tiles in flight (the next Q K^T is issued a tile ahead)
constexpr int kAVStages = 2;            // value tiles in flight
constexpr int kASplitMinTiles = 8;      // key tiles per unit from which two CTAs share a unit
constexpr float kALog2e = 1.4426950408889634f;

template <int D>
struct ASmem {
  static constexpr int kBoxes = D / 64;
  static constexpr int kBoxBytes = kATile * 128;
  static constexpr int kTileBytes = kBoxes * kBoxBytes;
  static constexpr int kQOff = 0;
  static constexpr int kKOff = kTileBytes;
  static constexpr int kVOff = kKOff + kAKStages * kTileBytes;
  static constexpr int kBarOff = kVOff + kAVStages * kTileBytes;
  static constexpr int kNumBars = 1 + 2 * kAKStages + 2 * kAVStages + 10;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  static constexpr int kMxOff = kMiscOff + 16;                             // float [2 warpgroups][128]: row references
  static constexpr int kLxOff = kMxOff + 2 * kATile * 4;                   // float [2 warpgroups][128]: row sums
  static constexpr int kBytes = kLxOff + 2 * kATile * 4;
  static constexpr int kDynamic = kBytes + 1024;
};

// The value operand V is row-major in shared memory (row = k index, 64 contiguous n per 128-byte row): an N-major
// descriptor with 128-byte swizzle - 8-row groups 1024 bytes apart along k, the next 64 columns one box away
// (that distance goes into the leading-byte-offset field of the low word).
// bf16 x bf16 -> fp32, A K-major (tensor memory), B N-major.
__device__ __forceinline__ uint32_t idesc_bf16_f32_bn(uint32_t m, uint32_t n) { return idesc_bf16_f32(m, n) | (1u << 16); }

__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* u) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]), "r"(u[8]),
        "r"(u[9]), "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15]), "r"(u[16]), "r"(u[17]),
        "r"(u[18]), "r"(u[19]), "r"(u[20]), "r"(u[21]), "r"(u[22]), "r"(u[23]), "r"(u[24]), "r"(u[25]), "r"(u[26]),
        "r"(u[27]), "r"(u[28]), "r"(u[29]), "r"(u[30]), "r"(u[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* u) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]), "r"(u[8]),
        "r"(u[9]), "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// Cluster-wide barrier, every thread of every CTA of the cluster once per phase (no convergence requirement);
// release / acquire order the distributed-shared-memory stores made before it against the loads after it.
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

struct ABars {
  uint64_t* qfull;
  uint64_t *kfull, *kempty;                    // [kAKStages]
  uint64_t *vfull, *vempty;                    // [kAVStages]
  uint64_t* sfull;                             // [2 buffers]
  uint64_t *pready, *odone;                    // [2 buffers][2 warpgroups]
};
__device__ __forceinline__ ABars carve_abars(uint8_t* base, int off) {
  uint64_t* b = reinterpret_cast<uint64_t*>(base + off);
  ABars r;
  r.qfull = b; r.kfull = b + 1; r.kempty = r.kfull + kAKStages; r.vfull = r.kempty + kAKStages; r.vempty = r.vfull + kAVStages;
  r.sfull = r.vempty + kAVStages; r.pready = r.sfull + 2; r.odone = r.pready + 4;
  return r;
}

// Tile j of the key walk: compacted rows first, then live rows.
struct ATile { bool cache; int row; int valid; };
__device__ __forceinline__ ATile a_tile(int j, int c0, int nc, int l0, int M) {
  const int TC = (nc + kATile - 1) / kATile;
  ATile t;
  t.cache = j < TC;
  const int off = (t.cache ? j : j - TC) * kATile;
  t.row = (t.cache ? c0 : l0) + off;
  t.valid = min(kATile, (t.cache ? nc : M) - off);
  return t;
}

// grid (q tiles, H, R)
template <int D>
__global__ void __launch_bounds__(AWgs<D>::kThreads, 1)
attend_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kl,
          const __grid_constant__ CUtensorMap map_vl, const __grid_constant__ CUtensorMap map_kc,
          const __grid_constant__ CUtensorMap map_vc, Shape sh, const int32_t* __restrict__ offsets,
          const int32_t* __restrict__ q_cu, int sum_q, __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
          uint32_t* __restrict__ status) {
  using S = ASmem<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const ABars bars = carve_abars(base, S::kBarOff);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + S::kMiscOff);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(base + S::kMiscOff + 4);

  // Set-up that touches no global memory runs before the wait for the previous kernel of the stream.
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(bars.qfull, 1);
    for (int s = 0; s < kAKStages; ++s) { mbar_init(bars.kfull + s, 1); mbar_init(bars.kempty + s, 1); }
    for (int s = 0; s < kAVStages; ++s) { mbar_init(bars.vfull + s, 1); mbar_init(bars.vempty + s, 2); }   // both P V issuers release a stage
    for (int b = 0; b < 2; ++b) {
      mbar_init(bars.sfull + b, 1);
      for (int w = 0; w < 2; ++w) { mbar_init(bars.pready + 2 * b + w, kATile); mbar_init(bars.odone + 2 * b + w, 1); }
    }
    *abort_flag = 0u;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) {                                  // kernel parameters: may be fetched before the wait
    prefetch_tmap(&map_q); prefetch_tmap(&map_kl); prefetch_tmap(&map_vl); prefetch_tmap(&map_kc); prefetch_tmap(&map_vc);
  }
  pdl_wait();

  // A cluster of `nsplit` CTAs (1 or 2) shares one (query tile, head): CTA `part` walks its contiguous share of
  // the key tiles; the partial (max, sum, output) of CTA 1 is merged into CTA 0's through distributed shared memory.
  cooperative_groups::cluster_group cluster = cooperative_groups::this_cluster();
  const int nsplit = (int)cluster.num_blocks(), part = (int)cluster.block_rank();
  const int qt = blockIdx.x / nsplit, h = blockIdx.y, r = blockIdx.z, hk = h / sh.g;
  const int seg = r * sh.Hkv + hk;
  // the four loads go out together (they are independent, and nothing can start before them)
  // q_cu = the query rows of every request: the live rows themselves (q_cu == live_cu), or the refreshed subset of them
  const int l0 = sh.live_cu[r], l1 = sh.live_cu[r + 1], c0 = offsets[seg], c1 = offsets[seg + 1];
  const int ql0 = q_cu[r], ql1 = q_cu[r + 1];
  const int M = l1 - l0, nc = c1 - c0, Mq = ql1 - ql0;
  const int q0 = qt * kATile;
  if (q0 >= Mq) {                                           // uniform over the block: nothing to do for this tile
    if (warp == 1) tmem_dealloc(tmem_base, 512);
    return;
  }
  const int nt_all = (nc + kATile - 1) / kATile + (M + kATile - 1) / kATile;
  const int per_part = (nt_all + nsplit - 1) / nsplit;
  const int j_first = part * per_part;                     // this CTA walks tiles [j_first, j_first + nt)
  const int nt = max(0, min(per_part, nt_all - j_first));

  const uint32_t tm_s = tmem_base, tm_o = tmem_base + 256;   // S/P buffers at columns 0 / 128, the warpgroups' outputs at 256 / 384

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(bars.qfull, S::kTileBytes);
      for (int b = 0; b < S::kBoxes; ++b) tma_load_3d(base + S::kQOff + b * S::kBoxBytes, &map_q, bars.qfull, b * 64, h, ql0 + q0);
      // two independent rings (keys, values): whichever has a free stage gets its next tile, keys first
      int jk = 0, jv = 0;
      const unsigned long long t_start = global_ns();
      uint32_t spins = 0;
      bool ok = true, prefetched = false;
      while (jk < nt || jv < nt) {
        bool issued = false;
        if (jk < nt) {
          const int stage = jk % kAKStages, use = jk / kAKStages;
          if (mbar_try_wait(bars.kempty + stage, (use & 1) ^ 1)) {
            const ATile t = a_tile(j_first + jk, c0, nc, l0, M);
            mbar_expect_tx(bars.kfull + stage, S::kTileBytes);
            for (int b = 0; b < S::kBoxes; ++b)
              tma_load_3d(base + S::kKOff + stage * S::kTileBytes + b * S::kBoxBytes, t.cache ? &map_kc : &map_kl,
                          bars.kfull + stage, b * 64, t.cache ? 0 : hk, t.row);
            ++jk;
            issued = true;
          }
        }
        if (jv < nt) {
          const int stage = jv % kAVStages, use = jv / kAVStages;
          if (mbar_try_wait(bars.vempty + stage, (use & 1) ^ 1)) {
            const ATile t = a_tile(j_first + jv, c0, nc, l0, M);
            mbar_expect_tx(bars.vfull + stage, S::kTileBytes);
            for (int b = 0; b < S::kBoxes; ++b)
              tma_load_3d(base + S::kVOff + stage * S::kTileBytes + b * S::kBoxBytes, t.cache ? &map_vc : &map_vl,
                          bars.vfull + stage, b * 64, t.cache ? 0 : hk, t.row);
            ++jv;
            issued = true;
          }
        }
        if (!prefetched && jk >= min(nt, kAKStages) && jv >= min(nt, kAVStages)) {
          // the rings are full: ask for the later tiles to be brought into L2, so that their ring loads pay L2 latency only
          for (int j = kAVStages; j < nt; ++j) {
            const ATile t = a_tile(j_first + j, c0, nc, l0, M);
            for (int b = 0; b < S::kBoxes; ++b) {
              if (j >= kAKStages) tma_prefetch_l2_3d(t.cache ? &map_kc : &map_kl, b * 64, t.cache ? 0 : hk, t.row);
              tma_prefetch_l2_3d(t.cache ? &map_vc : &map_vl, b * 64, t.cache ? 0 : hk, t.row);
            }
          }
          prefetched = true;
        }
        if (!issued && (++spins & 255u) == 0u) {             // bounded like every other wait
          if (*abort_flag) { ok = false; break; }
          if (global_ns() - t_start > kWaitLimitNs) {
            *abort_flag = 1u; atomicOr(status, (uint32_t)MASKKV_FLAG_TIMEOUT); atomicExch(status + 1, 0x301u);
            ok = false; break;
          }
        }
      }
      if (!ok) {   // wait (bounded) for the copies already issued
        for (int i = max(0, jk - kAKStages); i < jk; ++i)
          for (uint32_t it = 0; it < (1u << 20) && !mbar_try_wait(bars.kfull + i % kAKStages, (i / kAKStages) & 1); ++it) __nanosleep(64);
        for (int i = max(0, jv - kAVStages); i < jv; ++i)
          for (uint32_t it = 0; it < (1u << 20) && !mbar_try_wait(bars.vfull + i % kAVStages, (i / kAVStages) & 1); ++it) __nanosleep(64);
      }
    }
    if (nsplit > 1) { cluster_barrier(); cluster_barrier(); }   // the two phases of the merge below
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_bf16_f32(kATile, kATile);
      const uint32_t q_lo = smem_desc_lo(smem_u32(base + S::kQOff));
      bool ok = mbar_wait(bars.qfull, 0, abort_flag, status, 0x303);
      tc_fence_after();
      for (int j = 0; ok && j < nt; ++j) {
        const int b = j & 1, stage = j % kAKStages, use = j / kAKStages;
        if (!(ok = mbar_wait(bars.kfull + stage, use & 1, abort_flag, status, 0x304))) break;
        // S/P buffer b is free once both P V products of tile j - 2 have read P from it
        if (j >= 2) {
          if (!(ok = mbar_wait(bars.odone + 2 * b, ((j - 2) >> 1) & 1, abort_flag, status, 0x30b))) break;
          if (!(ok = mbar_wait(bars.odone + 2 * b + 1, ((j - 2) >> 1) & 1, abort_flag, status, 0x30c))) break;
        }
        tc_fence_after();
        const uint32_t k_lo = smem_desc_lo(smem_u32(base + S::kKOff + stage * S::kTileBytes));
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t o = ((kk >> 2) * S::kBoxBytes + (kk & 3) * 32) >> 4;
          umma_ss(tm_s + b * kATile, make_desc(q_lo + o, kDescHiSw128), make_desc(k_lo + o, kDescHiSw128), idesc_qk, kk > 0);
        }
        umma_commit(bars.sfull + b);
        umma_commit(bars.kempty + stage);
      }
    }
    if (nsplit > 1) { cluster_barrier(); cluster_barrier(); }
  } else if (warp >= AWgs<D>::kPvWarp) {
    // P V of warpgroup w: O_w += P[:, 64w .. 64w+63] V[64w .. 64w+63, :], four k-steps, accumulated in tensor memory
    // over all tiles (the warpgroup rescales O_w itself in the rare case its reference moves).
    const int w = warp - AWgs<D>::kPvWarp;
    if (lane == 0) {
      const uint32_t idesc_pv = idesc_bf16_f32_bn(kATile, D);
      bool ok = true;
      for (int j = 0; ok && j < nt; ++j) {
        const int b = j & 1, stage = j % kAVStages, use = j / kAVStages;
        if (!(ok = mbar_wait(bars.vfull + stage, use & 1, abort_flag, status, 0x305))) break;
        if (!(ok = mbar_wait(bars.pready + 2 * b + w, (j >> 1) & 1, abort_flag, status, 0x307))) break;
        tc_fence_after();
        // N-major descriptor: low word = address | (box stride between the two 64-column halves), high word as K-major
        const uint32_t v_lo = ((smem_u32(base + S::kVOff + stage * S::kTileBytes) & 0x3ffffu) >> 4) | ((uint32_t)(S::kBoxBytes >> 4) << 16);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          // P of keys [64w, 64w + 64) sits in packed columns [64w, 64w + 32) of the S/P buffer
          umma_ts(tm_o + w * kATile, tm_s + b * kATile + 64 * w + 8 * kk, make_desc(v_lo + (((4 * w + kk) * 16 * 128) >> 4), kDescHiSw128),
                  idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
        umma_commit(bars.odone + 2 * b + w);
        umma_commit(bars.vempty + stage);
      }
    }
    if (nsplit > 1) { cluster_barrier(); cluster_barrier(); }
  } else {
    // Two softmax warpgroups, each an online softmax of its own over "its" 64 keys of every tile: thread (wg, row)
    // owns S columns [64 wg, 64 wg + 64) of its query row, keeps its own reference m and sum l, writes P over the columns
    // it has just read, and its P V accumulates in the warpgroup's own output O_wg in tensor memory.  Nothing is
    // exchanged per tile, so the two groups drift apart and one's exponentials overlap the other's tensor-memory
    // traffic.  m only moves when a logit exceeds it by more than 2^kSlack (P <= 2^kSlack is harmless in bf16 and
    // fp32); then the thread rescales its row of O_wg in tensor memory.  The groups meet once, after the last tile.
    constexpr int NW = AWgs<D>::kNW;
    constexpr int SC = kATile / NW;                         // 64 key columns of a tile per thread
    constexpr float kSlack = 8.f;
    const int wg = (warp - 2) >> 2;
    const int lane_group = warp & 3;
    const int row = lane_group * 32 + lane;                 // query inside the tile
    const int tid_all = wg * kATile + ((warp - 2) & 3) * 32 + lane;   // 0 .. 255 over the softmax warpgroups
    const uint32_t lane_addr = (uint32_t)(lane_group * 32) << 16;
    const uint32_t o_addr = tm_o + lane_addr + wg * kATile;  // this row of O_wg
    const float cs = sh.scale * kALog2e;
    float* mx = reinterpret_cast<float*>(base + S::kMxOff);
    float* lx = reinterpret_cast<float*>(base + S::kLxOff);
    constexpr int OC = D / NW;                              // output columns per thread after the groups have met
    float m = -INFINITY, l = 0.f;
    bool ok = true;

    // After a failed wait a thread skips the tensor-memory work but still reaches every named barrier.
    for (int j = 0; j < nt; ++j) {
      const int b = j & 1;
      const ATile t = a_tile(j_first + j, c0, nc, l0, M);
      const int my_valid = min(SC, max(0, t.valid - wg * SC));   // valid columns among this thread's 64
      if (ok && t.valid < kATile) {
        // ragged tail: zero the value rows that do not belong to this tile.  Each warpgroup clears all of them (its
        // own P V is released by its own threads only, so it may not rely on the other group's stores).
        const int stage = j % kAVStages, su = j / kAVStages;
        if ((ok = mbar_wait(bars.vfull + stage, su & 1, abort_flag, status, 0x309))) {
          uint8_t* v_tile = base + S::kVOff + stage * S::kTileBytes;
          const int n16 = (kATile - t.valid) * 8;           // 16-byte pieces per box
          for (int bx = 0; bx < S::kBoxes; ++bx) {
            uint4* dst = reinterpret_cast<uint4*>(v_tile + bx * S::kBoxBytes + t.valid * 128);
            for (int e = tid_all & (kATile - 1); e < n16; e += kATile) dst[e] = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_async_smem();
        }
      }
      if (ok) ok = mbar_wait(bars.sfull + b, (j >> 1) & 1, abort_flag, status, 0x30a);
      ok = __all_sync(0xffffffffu, ok);                     // the tensor-memory instructions below are warp-wide
      if (!ok) continue;
      tc_fence_after();
      const uint32_t s_addr = tm_s + lane_addr + b * kATile + wg * SC;
      float v[SC];                                          // the thread's logits, read once
#pragma unroll
      for (int cb = 0; cb < SC / 32; ++cb) tmem_ld32(s_addr + cb * 32, v + cb * 32);
      tmem_ld_wait();
      if (my_valid < SC) {                                   // masked columns of a ragged tile do not take part
#pragma unroll
        for (int c = 0; c < SC; ++c) if (c >= my_valid) v[c] = -INFINITY;
      }
      float tmax = -INFINITY;
#pragma unroll
      for (int c = 0; c < SC; c += 2) tmax = max3(tmax, v[c], v[c + 1]);
      // The reference moves up when a logit exceeds it by more than 2^kSlack: the sum and this row of O_wg are rescaled,
      // once the previous tile's P V has landed.  Tensor-memory loads and stores are warp-wide instructions, so the whole
      // warp goes through them as soon as one row needs it (factor 1 for the others).
      const bool grow = m != -INFINITY && (tmax - m) * cs > kSlack;
      const float f = grow ? ex2((m - tmax) * cs) : 1.f;
      if (__any_sync(0xffffffffu, grow)) {
        ok = __all_sync(0xffffffffu, mbar_wait(bars.odone + 2 * ((j - 1) & 1) + wg, ((j - 1) >> 1) & 1, abort_flag, status, 0x308));
        if (ok) {
          tc_fence_after();
#pragma unroll
          for (int cb = 0; cb < D / 32; ++cb) {
            float ov[32];
            tmem_ld32(o_addr + cb * 32, ov);
            tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 32; ++c) ov[c] *= f;
            tmem_st32(o_addr + cb * 32, reinterpret_cast<const uint32_t*>(ov));
          }
          tmem_st_wait();
        }
      }
      if (grow) { l *= f; m = tmax; }
      else if (m == -INFINITY) m = tmax;                    // nothing accumulated so far (O_wg is zero or not yet written)
      if (!ok) continue;
      // P = 2^(s*c - m*c) as bf16 pairs (a masked column gives 2^-inf = 0), written over the columns just read
      uint32_t packed[SC / 2];
      float rs = 0.f;
      if (m == -INFINITY) {                                  // not a single valid column yet: P = 0
#pragma unroll
        for (int c = 0; c < SC / 2; ++c) packed[c] = 0u;
      } else {
        const float neg = -m * cs;
#pragma unroll
        for (int c = 0; c < SC; c += 2) {
          const float p0 = ex2(fmaf(v[c], cs, neg)), p1 = ex2(fmaf(v[c + 1], cs, neg));
          rs += p0 + p1;
          packed[c / 2] = pack_bf16(p0, p1);
        }
      }
      tmem_st32(s_addr, packed);
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(bars.pready + 2 * b + wg);
      l += rs;
    }
    // The groups meet: common reference, total sum, and both groups' O scaled onto the common reference.  Thread
    // (wg, row) ends up with output columns [OC wg, OC wg + OC) of its row; its row of BOTH accumulators sits in
    // tensor-memory lanes the thread may read, so only the references and sums go through shared memory.
    if (nt > 0) {                                            // both streams' last P V must have landed
      if (ok) ok = mbar_wait(bars.odone + 2 * ((nt - 1) & 1), ((nt - 1) >> 1) & 1, abort_flag, status, 0x30d);
      if (ok) ok = mbar_wait(bars.odone + 2 * ((nt - 1) & 1) + 1, ((nt - 1) >> 1) & 1, abort_flag, status, 0x30e);
    }
    ok = __all_sync(0xffffffffu, ok);
    if (ok) tc_fence_after();
    mx[wg * kATile + row] = m;
    lx[wg * kATile + row] = l;
    named_barrier(1, NW * kATile);
    const float m_other = mx[(wg ^ 1) * kATile + row], l_other = lx[(wg ^ 1) * kATile + row];
    const float m_all = fmaxf(m, m_other);
    const float a_me = m == -INFINITY ? 0.f : ex2((m - m_all) * cs);
    const float a_other = m_other == -INFINITY ? 0.f : ex2((m_other - m_all) * cs);
    const float a_of[2] = {wg == 0 ? a_me : a_other, wg == 0 ? a_other : a_me};   // scale of stream 0, stream 1
    float o[OC];
#pragma unroll
    for (int c = 0; c < OC; ++c) o[c] = 0.f;
    if (ok && nt > 0) {                                      // warp-uniform; a stream that never saw a valid key holds exact zeros
#pragma unroll
      for (int w2 = 0; w2 < NW; ++w2) {
#pragma unroll
        for (int cb = 0; cb < OC / 32; ++cb) {
          float ov[32];
          tmem_ld32(tm_o + lane_addr + w2 * kATile + wg * OC + cb * 32, ov);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[cb * 32 + c] = fmaf(ov[c], a_of[w2], o[cb * 32 + c]);
        }
      }
    }
    l = l * a_me + l_other * a_other;
    m = m_all;
    if (nsplit > 1) {
      // Exchange area in CTA 0: its key ring, free once both CTAs have finished their tiles (first barrier).
      // xo4[column group of 4][row] as float4 (a warp's 32 rows of a group are 512 contiguous bytes, for the remote
      // stores as for the loads), then xm[row], xl[row].
      float4* xo4 = reinterpret_cast<float4*>(base + S::kKOff);
      float* xm = reinterpret_cast<float*>(xo4 + (D / 4) * kATile);
      float* xl = xm + kATile;
      cluster_barrier();
      if (part == 1) {
        float4* ro = cluster.map_shared_rank(xo4, 0) + (wg * OC / 4) * kATile + row;
#pragma unroll
        for (int c = 0; c < OC; c += 4) ro[(c / 4) * kATile] = make_float4(o[c], o[c + 1], o[c + 2], o[c + 3]);
        if (wg == 0) { cluster.map_shared_rank(xm, 0)[row] = m; cluster.map_shared_rank(xl, 0)[row] = l; }
      }
      cluster_barrier();
      if (part == 0) {
        const float m1 = xm[row], l1 = xl[row];
        const float m_all = fmaxf(m, m1);
        const float a0 = ex2((m - m_all) * cs), a1 = ex2((m1 - m_all) * cs);   // an empty share has m1 = -inf: a1 = 0
        l = l * a0 + l1 * a1;
        const float4* po = xo4 + (wg * OC / 4) * kATile + row;
#pragma unroll
        for (int c = 0; c < OC; c += 4) {
          const float4 v4 = po[(c / 4) * kATile];
          o[c] = o[c] * a0 + v4.x * a1; o[c + 1] = o[c + 1] * a0 + v4.y * a1;
          o[c + 2] = o[c + 2] * a0 + v4.z * a1; o[c + 3] = o[c + 3] * a0 + v4.w * a1;
        }
        m = m_all;
      }
    }
    // Output: a thread holds D/NW columns of one row, which would make every store instruction touch 32 rows.  The
    // tile goes through shared memory instead (the value ring, free now; rows padded by 16 bytes against bank
    // conflicts) and leaves as whole 2*D-byte rows, 16 bytes per lane.
    const int i = q0 + row;
    uint8_t* stage_o = base + S::kVOff;
    constexpr int RS = D * 2 + 16;
    if (ok && part == 0) {
      const float inv = 1.f / l;
      uint4* dst = reinterpret_cast<uint4*>(stage_o + row * RS + wg * OC * 2);
#pragma unroll
      for (int c = 0; c < OC; c += 8) {
        uint4 w;
        w.x = pack_bf16(o[c] * inv, o[c + 1] * inv);
        w.y = pack_bf16(o[c + 2] * inv, o[c + 3] * inv);
        w.z = pack_bf16(o[c + 4] * inv, o[c + 5] * inv);
        w.w = pack_bf16(o[c + 6] * inv, o[c + 7] * inv);
        dst[c / 8] = w;
      }
      if (wg == 0 && lse != nullptr && i < Mq && !*abort_flag) lse[(long long)h * sum_q + ql0 + i] = m * sh.scale + logf(l);
    }
    named_barrier(1, NW * kATile);
    if (part == 0 && !*abort_flag) {
      constexpr int PPR = D * 2 / 16;                        // 16-byte pieces per row
      const int pieces = min(kATile, Mq - q0) * PPR;
      uint8_t* out_tile = reinterpret_cast<uint8_t*>(out + (long long)(ql0 + q0) * sh.q_ts + (long long)h * sh.q_hs);
      for (int e = tid_all; e < pieces; e += NW * kATile) {
        const int rr = e / PPR, pc = e % PPR;
        *reinterpret_cast<uint4*>(out_tile + (long long)rr * sh.q_ts * 2 + pc * 16) =
            *reinterpret_cast<const uint4*>(stage_o + rr * RS + pc * 16);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

// =====================================================================================================
// Two query tiles per CTA, for launches with (many) more units than SMs - batches of requests or layers.
//
// A unit is a (128-query tile, query head) of one request; two units that share a KV head - the two query tiles of a
// head, or tiles of different query heads of one group - walk the same key / value tiles, so one CTA takes both: the
// tiles are fetched once, and while the softmax warpgroup of one unit exponentiates, the tensor cores work on the
// other unit's products.  Stream w (0 / 1): its logits S_w and, over them, its P in tensor-memory columns
// [128 w, 128 w + 128), its output O_w in [256 + 128 w, 384 + 128 w); softmax warpgroup w owns the stream (thread =
// query row, all 128 key columns of a tile in two halves of 64, reference moved lazily as above); P V of stream w is
// issued by warp 10 + w, both Q K^T by warp 1.  S_w is single-buffered: Q K^T of tile j + 1 of a stream follows its
// P V of tile j, and the other stream's work fills the tensor pipe meanwhile.  No merge at the end: a warpgroup
// normalises and stores its own tile.  grid (pairs of units per KV head, H_kv, R).
// =====================================================================================================
constexpr int kPKStages = 2;
constexpr int kPVStages = 2;

template <int D>
struct PSmem {
  static constexpr int kBoxes = D / 64;
  static constexpr int kBoxBytes = kATile * 128;
  static constexpr int kTileBytes = kBoxes * kBoxBytes;
  static constexpr int kQOff = 0;                                          // two query tiles
  static constexpr int kKOff = 2 * kTileBytes;
  static constexpr int kVOff = kKOff + kPKStages * kTileBytes;
  static constexpr int kBarOff = kVOff + kPVStages * kTileBytes;
  static constexpr int kNumBars = 1 + 2 * kPKStages + 2 * kPVStages + 6;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  static constexpr int kBytes = kMiscOff + 16;
  static constexpr int kDynamic = kBytes + 1024;
};

struct PBars {
  uint64_t* qfull;
  uint64_t *kfull, *kempty;                    // [kPKStages]
  uint64_t *vfull, *vempty;                    // [kPVStages]
  uint64_t *sfull, *pready, *odone;            // [2 streams]
};
__device__ __forceinline__ PBars carve_pbars(uint8_t* base, int off) {
  uint64_t* b = reinterpret_cast<uint64_t*>(base + off);
  PBars r;
  r.qfull = b; r.kfull = b + 1; r.kempty = r.kfull + kPKStages; r.vfull = r.kempty + kPKStages; r.vempty = r.vfull + kPVStages;
  r.sfull = r.vempty + kPVStages; r.pready = r.sfull + 2; r.odone = r.pready + 2;
  return r;
}

template <int D>
__global__ void __launch_bounds__(AWgs<D>::kThreads, 1)
attend_pair_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kl,
               const __grid_constant__ CUtensorMap map_vl, const __grid_constant__ CUtensorMap map_kc,
               const __grid_constant__ CUtensorMap map_vc, Shape sh, const int32_t* __restrict__ offsets,
               const int32_t* __restrict__ q_cu, int sum_q, int q_tiles, __nv_bfloat16* __restrict__ out,
               float* __restrict__ lse, uint32_t* __restrict__ status) {
  using S = PSmem<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const PBars bars = carve_pbars(base, S::kBarOff);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base + S::kMiscOff);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(base + S::kMiscOff + 4);

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(bars.qfull, 1);
    for (int st = 0; st < kPKStages; ++st) { mbar_init(bars.kfull + st, 1); mbar_init(bars.kempty + st, 1); }
    for (int st = 0; st < kPVStages; ++st) { mbar_init(bars.vfull + st, 1); mbar_init(bars.vempty + st, 2); }   // both P V issuers release a stage
    for (int w = 0; w < 2; ++w) { mbar_init(bars.sfull + w, 1); mbar_init(bars.pready + w, kATile); mbar_init(bars.odone + w, 1); }
    *abort_flag = 0u;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) {
    prefetch_tmap(&map_q); prefetch_tmap(&map_kl); prefetch_tmap(&map_vl); prefetch_tmap(&map_kc); prefetch_tmap(&map_vc);
  }
  pdl_wait();

  const int hk = blockIdx.y, r = blockIdx.z;
  const int seg = r * sh.Hkv + hk;
  const int l0 = sh.live_cu[r], l1 = sh.live_cu[r + 1], c0 = offsets[seg], c1 = offsets[seg + 1];
  const int ql0 = q_cu[r], ql1 = q_cu[r + 1];
  const int M = l1 - l0, nc = c1 - c0, Mq = ql1 - ql0;
  // the two units of this CTA: unit u of the KV head = (query head hk*g + u / q_tiles, query tile u % q_tiles)
  int uh[2], uq0[2];
  bool active[2];
#pragma unroll
  for (int w = 0; w < 2; ++w) {
    const int u = 2 * (int)blockIdx.x + w;
    uh[w] = hk * sh.g + u / q_tiles;
    uq0[w] = (u % q_tiles) * kATile;
    active[w] = u < sh.g * q_tiles && uq0[w] < Mq;
  }
  if (!active[0] && !active[1]) {                           // uniform over the block
    if (warp == 1) tmem_dealloc(tmem_base, 512);
    return;
  }
  const int nt = (nc + kATile - 1) / kATile + (M + kATile - 1) / kATile;
  const uint32_t tm_s = tmem_base, tm_o = tmem_base + 256;

  if (warp == 0) {
    if (lane == 0) {
      const int n_act = (active[0] ? 1 : 0) + (active[1] ? 1 : 0);
      mbar_expect_tx(bars.qfull, n_act * S::kTileBytes);
      for (int w = 0; w < 2; ++w)
        if (active[w])
          for (int b = 0; b < S::kBoxes; ++b)
            tma_load_3d(base + S::kQOff + w * S::kTileBytes + b * S::kBoxBytes, &map_q, bars.qfull, b * 64, uh[w], ql0 + uq0[w]);
      int jk = 0, jv = 0;
      const unsigned long long t_start = global_ns();
      uint32_t spins = 0;
      bool ok = true;
      while (jk < nt || jv < nt) {
        bool issued = false;
        if (jk < nt) {
          const int stage = jk % kPKStages, use = jk / kPKStages;
          if (mbar_try_wait(bars.kempty + stage, (use & 1) ^ 1)) {
            const ATile t = a_tile(jk, c0, nc, l0, M);
            mbar_expect_tx(bars.kfull + stage, S::kTileBytes);
            for (int b = 0; b < S::kBoxes; ++b)
              tma_load_3d(base + S::kKOff + stage * S::kTileBytes + b * S::kBoxBytes, t.cache ? &map_kc : &map_kl,
                          bars.kfull + stage, b * 64, t.cache ? 0 : hk, t.row);
            ++jk;
            issued = true;
          }
        }
        if (jv < nt) {
          const int stage = jv % kPVStages, use = jv / kPVStages;
          if (mbar_try_wait(bars.vempty + stage, (use & 1) ^ 1)) {
            const ATile t = a_tile(jv, c0, nc, l0, M);
            mbar_expect_tx(bars.vfull + stage, S::kTileBytes);
            for (int b = 0; b < S::kBoxes; ++b)
              tma_load_3d(base + S::kVOff + stage * S::kTileBytes + b * S::kBoxBytes, t.cache ? &map_vc : &map_vl,
                          bars.vfull + stage, b * 64, t.cache ? 0 : hk, t.row);
            ++jv;
            issued = true;
          }
        }
        if (!issued && (++spins & 255u) == 0u) {             // bounded like every other wait
          if (*abort_flag) { ok = false; break; }
          if (global_ns() - t_start > kWaitLimitNs) {
            *abort_flag = 1u; atomicOr(status, (uint32_t)MASKKV_FLAG_TIMEOUT); atomicExch(status + 1, 0x321u);
            ok = false; break;
          }
        }
      }
      if (!ok) {   // wait (bounded) for the copies already issued
        for (int i = max(0, jk - kPKStages); i < jk; ++i)
          for (uint32_t it = 0; it < (1u << 20) && !mbar_try_wait(bars.kfull + i % kPKStages, (i / kPKStages) & 1); ++it) __nanosleep(64);
        for (int i = max(0, jv - kPVStages); i < jv; ++i)
          for (uint32_t it = 0; it < (1u << 20) && !mbar_try_wait(bars.vfull + i % kPVStages, (i / kPVStages) & 1); ++it) __nanosleep(64);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_bf16_f32(kATile, kATile);
      bool ok = mbar_wait(bars.qfull, 0, abort_flag, status, 0x323);
      tc_fence_after();
      for (int j = 0; ok && j < nt; ++j) {
        const int stage = j % kPKStages, use = j / kPKStages;
        if (!(ok = mbar_wait(bars.kfull + stage, use & 1, abort_flag, status, 0x324))) break;
        const uint32_t k_lo = smem_desc_lo(smem_u32(base + S::kKOff + stage * S::kTileBytes));
        for (int w = 0; w < 2 && ok; ++w) {
          if (!active[w]) continue;
          // S_w is free once P V of tile j - 1 of this stream has read P from it
          if (j >= 1 && !(ok = mbar_wait(bars.odone + w, (j - 1) & 1, abort_flag, status, 0x32b))) break;
          tc_fence_after();
          const uint32_t q_lo = smem_desc_lo(smem_u32(base + S::kQOff + w * S::kTileBytes));
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t o = ((kk >> 2) * S::kBoxBytes + (kk & 3) * 32) >> 4;
            umma_ss(tm_s + w * kATile, make_desc(q_lo + o, kDescHiSw128), make_desc(k_lo + o, kDescHiSw128), idesc_qk, kk > 0);
          }
          umma_commit(bars.sfull + w);
        }
        umma_commit(bars.kempty + stage);
      }
    }
  } else if (warp >= AWgs<D>::kPvWarp) {
    // P V of stream w: O_w += P_w V over the tile's 128 keys, eight k-steps, accumulated in tensor memory over all tiles
    const int w = warp - AWgs<D>::kPvWarp;
    if (lane == 0) {
      const uint32_t idesc_pv = idesc_bf16_f32_bn(kATile, D);
      bool ok = true;
      for (int j = 0; ok && j < nt; ++j) {
        const int stage = j % kPVStages, use = j / kPVStages;
        if (!(ok = mbar_wait(bars.vfull + stage, use & 1, abort_flag, status, 0x325))) break;
        if (active[w]) {
          if (!(ok = mbar_wait(bars.pready + w, j & 1, abort_flag, status, 0x327))) break;
          tc_fence_after();
          const uint32_t v_lo = ((smem_u32(base + S::kVOff + stage * S::kTileBytes) & 0x3ffffu) >> 4) | ((uint32_t)(S::kBoxBytes >> 4) << 16);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            // P of keys [16 kk, 16 kk + 16) sits in packed columns [8 kk, 8 kk + 8) of S_w
            umma_ts(tm_o + w * kATile, tm_s + w * kATile + 8 * kk, make_desc(v_lo + ((kk * 16 * 128) >> 4), kDescHiSw128), idesc_pv,
                    (j > 0 || kk > 0) ? 1u : 0u);
          umma_commit(bars.odone + w);
        }
        umma_commit(bars.vempty + stage);                    // an idle stream releases the stage at once
      }
    }
  } else {
    constexpr int SC = 64;                                  // key columns per half
    constexpr float kSlack = 8.f;
    const int w = (warp - 2) >> 2;                          // this warpgroup's stream
    const int lane_group = warp & 3;
    const int row = lane_group * 32 + lane;                 // query inside the tile
    const int tid_wg = ((warp - 2) & 3) * 32 + lane;        // 0 .. 127 inside the warpgroup
    const uint32_t lane_addr = (uint32_t)(lane_group * 32) << 16;
    const uint32_t s_addr = tm_s + lane_addr + w * kATile;
    const uint32_t o_addr = tm_o + lane_addr + w * kATile;
    const float cs = sh.scale * kALog2e;
    float m = -INFINITY, l = 0.f;
    bool ok = true;
    const bool mine = active[w];
    for (int j = 0; j < nt && mine; ++j) {
      const ATile t = a_tile(j, c0, nc, l0, M);
      if (ok && t.valid < kATile) {
        // ragged tail: zero the value rows that do not belong to this tile (each warpgroup clears all of them: its own
        // P V is released by its own threads only)
        const int stage = j % kPVStages, su = j / kPVStages;
        if ((ok = mbar_wait(bars.vfull + stage, su & 1, abort_flag, status, 0x329))) {
          uint8_t* v_tile = base + S::kVOff + stage * S::kTileBytes;
          const int n16 = (kATile - t.valid) * 8;
          for (int bx = 0; bx < S::kBoxes; ++bx) {
            uint4* dst = reinterpret_cast<uint4*>(v_tile + bx * S::kBoxBytes + t.valid * 128);
            for (int e = tid_wg; e < n16; e += kATile) dst[e] = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_async_smem();
        }
      }
      if (ok) ok = mbar_wait(bars.sfull + w, j & 1, abort_flag, status, 0x32a);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) continue;
      tc_fence_after();
      // Both halves of the tile feed one P V product, so they share one reference: a first pass over the logits finds the
      // row maximum, a second one (the logits are read from tensor memory again, which costs little) forms P.
      float tmax = -INFINITY;
#pragma unroll 1
      for (int hf = 0; hf < 2; ++hf) {
        const int my_valid = min(SC, max(0, t.valid - hf * SC));
        if (my_valid == 0) continue;                         // warp-uniform
        float v[SC];
#pragma unroll
        for (int cb = 0; cb < SC / 32; ++cb) tmem_ld32(s_addr + hf * SC + cb * 32, v + cb * 32);
        tmem_ld_wait();
        if (my_valid < SC) {
#pragma unroll
          for (int c = 0; c < SC; ++c) if (c >= my_valid) v[c] = -INFINITY;
        }
#pragma unroll
        for (int c = 0; c < SC; c += 2) tmax = max3(tmax, v[c], v[c + 1]);
      }
      // lazily moved reference: this stream's P V of tile j - 1 landed before Q K^T of tile j was issued, so O_w is at rest
      const bool grow = m != -INFINITY && (tmax - m) * cs > kSlack;
      const float f = grow ? ex2((m - tmax) * cs) : 1.f;
      if (j > 0 && __any_sync(0xffffffffu, grow)) {
#pragma unroll
        for (int cb = 0; cb < D / 32; ++cb) {
          float ov[32];
          tmem_ld32(o_addr + cb * 32, ov);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c) ov[c] *= f;
          tmem_st32(o_addr + cb * 32, reinterpret_cast<const uint32_t*>(ov));
        }
        tmem_st_wait();
      }
      if (grow) { l *= f; m = tmax; }
      else if (m == -INFINITY) m = tmax;
      float rs = 0.f;
      const float neg = -m * cs;
#pragma unroll 1
      for (int hf = 0; hf < 2; ++hf) {
        const int my_valid = min(SC, max(0, t.valid - hf * SC));
        uint32_t packed[SC / 2];
        if (my_valid == 0) {                                 // warp-uniform: a half without keys
#pragma unroll
          for (int c = 0; c < SC / 2; ++c) packed[c] = 0u;
        } else {
          float v[SC];
#pragma unroll
          for (int cb = 0; cb < SC / 32; ++cb) tmem_ld32(s_addr + hf * SC + cb * 32, v + cb * 32);
          tmem_ld_wait();
          if (my_valid < SC) {
#pragma unroll
            for (int c = 0; c < SC; ++c) if (c >= my_valid) v[c] = -INFINITY;
          }
#pragma unroll
          for (int c = 0; c < SC; c += 2) {
            const float p0 = ex2(fmaf(v[c], cs, neg)), p1 = ex2(fmaf(v[c + 1], cs, neg));
            rs += p0 + p1;
            packed[c / 2] = pack_bf16(p0, p1);
          }
        }
        // P of this half over logits that have been read: packed columns [32 hf, 32 hf + 32) of S_w.  (Half 1's logits
        // sit in columns 64 .. 127 and are read before anything is stored there.)
        tmem_st32(s_addr + hf * (SC / 2), packed);
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(bars.pready + w);
      l += rs;
    }
    // the stream's last P V must have landed
    if (mine && nt > 0 && ok) ok = mbar_wait(bars.odone + w, (nt - 1) & 1, abort_flag, status, 0x32d);
    ok = __all_sync(0xffffffffu, ok);
    named_barrier(3, 2 * kATile);                            // ... and the other stream's: nothing reads the rings any more
    if (mine) {
      // every other role has finished with shared memory by now (this stream's last P V read the last value tile, and the
      // key tiles were consumed before it): the tile leaves through the key ring (stream 0) / value ring (stream 1) as
      // whole 2*D-byte rows, 16 bytes per lane
      uint8_t* stage_o = base + (w == 0 ? S::kKOff : S::kVOff);
      constexpr int RS = D * 2 + 16;
      const int i = uq0[w] + row;
      if (ok) {
        tc_fence_after();
        const float inv = nt > 0 ? 1.f / l : 0.f;
#pragma unroll
        for (int cb = 0; cb < D / 32; ++cb) {
          float ov[32];
          if (nt > 0) { tmem_ld32(o_addr + cb * 32, ov); tmem_ld_wait(); }
          else {
#pragma unroll
            for (int c = 0; c < 32; ++c) ov[c] = 0.f;
          }
          uint4* dst = reinterpret_cast<uint4*>(stage_o + row * RS + cb * 64);
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            uint4 o4;
            o4.x = pack_bf16(ov[c] * inv, ov[c + 1] * inv);
            o4.y = pack_bf16(ov[c + 2] * inv, ov[c + 3] * inv);
            o4.z = pack_bf16(ov[c + 4] * inv, ov[c + 5] * inv);
            o4.w = pack_bf16(ov[c + 6] * inv, ov[c + 7] * inv);
            dst[c / 8] = o4;
          }
        }
        if (lse != nullptr && i < Mq && !*abort_flag) lse[(long long)uh[w] * sum_q + ql0 + i] = m * sh.scale + logf(l);
      }
      named_barrier(1 + w, kATile);
      if (!*abort_flag) {
        constexpr int PPR = D * 2 / 16;
        const int pieces = min(kATile, Mq - uq0[w]) * PPR;
        uint8_t* out_tile = reinterpret_cast<uint8_t*>(out + (long long)(ql0 + uq0[w]) * sh.q_ts + (long long)uh[w] * sh.q_hs);
        for (int e = tid_wg; e < pieces; e += kATile) {
          const int rr = e / PPR, pc = e % PPR;
          *reinterpret_cast<uint4*>(out_tile + (long long)rr * sh.q_ts * 2 + pc * 16) =
              *reinterpret_cast<const uint4*>(stage_o + rr * RS + pc * 16);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

namespace {
// The opt-in shared-memory size is an attribute of the kernel on ONE device: remembered per device, set with that device
// current (the entry points hold a device guard).
template <int D>
cudaError_t set_attend_attr(int device) {
  static bool done[kMaxAttrDevices] = {};
  if (device < 0 || device >= kMaxAttrDevices) return cudaErrorInvalidDevice;
  if (done[device]) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(attend_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, ASmem<D>::kDynamic);
  done[device] = e == cudaSuccess;
  return e;
}
template <int D>
cudaError_t set_attend_pair_attr(int device) {
  static bool done[kMaxAttrDevices] = {};
  if (device < 0 || device >= kMaxAttrDevices) return cudaErrorInvalidDevice;
  if (done[device]) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(attend_pair_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, PSmem<D>::kDynamic);
  done[device] = e == cudaSuccess;
  return e;
}
}  // namespace

bool attend_tc_supported(const maskkv_ctx* ctx, const Shape& sh) {
  return sh.dtype == MASKKV_BF16 && ctx->encode_tiled != nullptr && sh.sumM > 0 && ctx->smem_optin >= ASmem<128>::kDynamic;
}

int launch_attend_tc(maskkv_ctx* ctx, const Shape& sh, const void* q, const int32_t* q_cu, int sum_q, int max_q, const void* kl,
                     const void* vl, const void* kc, const void* vc, long long cache_rows, const int32_t* offsets, void* out,
                     float* lse, cudaStream_t st) {
  CUtensorMap mq, mkl, mvl, mkc, mvc;
  // an empty cache still needs valid maps: point them at the live tensors (no tile of them is ever requested)
  const void* kc_base = cache_rows > 0 && kc ? kc : kl;
  const void* vc_base = cache_rows > 0 && vc ? vc : vl;
  const uint64_t rows = cache_rows > 0 ? (uint64_t)cache_rows : 1;
  const bool ok = make_tmap_rows(ctx->encode_tiled, &mq, q, sh.d, sh.H, (uint64_t)sum_q, sh.q_hs * 2, sh.q_ts * 2, kATile) &&
                  make_tmap_rows(ctx->encode_tiled, &mkl, kl, sh.d, sh.Hkv, sh.sumM, sh.kv_hs * 2, sh.kv_ts * 2, kATile) &&
                  make_tmap_rows(ctx->encode_tiled, &mvl, vl, sh.d, sh.Hkv, sh.sumM, sh.kv_hs * 2, sh.kv_ts * 2, kATile) &&
                  make_tmap_rows(ctx->encode_tiled, &mkc, kc_base, sh.d, 1, rows, (uint64_t)sh.d * 2, (uint64_t)sh.d * 2, kATile) &&
                  make_tmap_rows(ctx->encode_tiled, &mvc, vc_base, sh.d, 1, rows, (uint64_t)sh.d * 2, (uint64_t)sh.d * 2, kATile);
  if (!ok) return 1;
  // Few (query tile, head, request) units leave most SMs idle and every CTA with a long chain of dependent tiles:
  // then two CTAs share a unit (cluster of 2 along x).  The merge costs about as much as three tiles (64 KB through
  // distributed shared memory), so the split only pays for long chains - eight tiles or more at the mean segment
  // length the capacity allows; with enough units it only adds set-up cost.
  const unsigned q_tiles = (unsigned)((max_q + kATile - 1) / kATile);
  const long long units = (long long)q_tiles * sh.H * sh.R;
  // Many more units than SMs (a batch of requests or layers): two units that share a KV head per CTA - their key / value
  // tiles are fetched once and the two softmax streams keep the tensor cores and the special-function unit busy in
  // turn.  Few units: one per CTA, so that all of them run at once (the per-layer latency case).
  const bool pairs_possible = sh.g * q_tiles >= 2;
  const bool want_pairs = (ctx->kernel_choice & 32u) ? true : (ctx->kernel_choice & 64u) ? false : units >= 2LL * ctx->sm_count;
  if (pairs_possible && want_pairs) {
    dim3 grid_p((sh.g * q_tiles + 1) / 2, sh.Hkv, sh.R);
    cudaError_t le;
    if (sh.d == 128) {
      if (set_attend_pair_attr<128>(ctx->device) != cudaSuccess) return 1;
      le = launch_overlapped(attend_pair_tc<128>, grid_p, dim3(AWgs<128>::kThreads), PSmem<128>::kDynamic, st, mq, mkl, mvl, mkc, mvc, sh,
                             offsets, q_cu, sum_q, (int)q_tiles, (__nv_bfloat16*)out, lse, ctx->status_dev);
    } else {
      if (set_attend_pair_attr<64>(ctx->device) != cudaSuccess) return 1;
      le = launch_overlapped(attend_pair_tc<64>, grid_p, dim3(AWgs<64>::kThreads), PSmem<64>::kDynamic, st, mq, mkl, mvl, mkc, mvc, sh,
                             offsets, q_cu, sum_q, (int)q_tiles, (__nv_bfloat16*)out, lse, ctx->status_dev);
    }
    if (le != cudaSuccess) { cudaGetLastError(); return 1; }
    return 0;
  }
  const long long mean_rows = cache_rows / ((long long)sh.R * sh.Hkv);
  const long long chain = (mean_rows + kATile - 1) / kATile + (sh.maxM + kATile - 1) / kATile;
  const unsigned nsplit = (2 * units <= ctx->sm_count && chain >= kASplitMinTiles) ? 2u : 1u;
  dim3 grid(q_tiles * nsplit, sh.H, sh.R);
  cudaError_t le;
  if (sh.d == 128) {
    if (set_attend_attr<128>(ctx->device) != cudaSuccess) return 1;
    le = launch_overlapped_cluster(attend_tc<128>, grid, dim3(AWgs<128>::kThreads), ASmem<128>::kDynamic, st, nsplit, mq, mkl, mvl, mkc, mvc,
                                  sh, offsets, q_cu, sum_q, (__nv_bfloat16*)out, lse, ctx->status_dev);
  } else {
    if (set_attend_attr<64>(ctx->device) != cudaSuccess) return 1;
    le = launch_overlapped_cluster(attend_tc<64>, grid, dim3(AWgs<64>::kThreads), ASmem<64>::kDynamic, st, nsplit, mq, mkl, mvl, mkc, mvc,
                                  sh, offsets, q_cu, sum_q, (__nv_bfloat16*)out, lse, ctx->status_dev);
  }
  if (le != cudaSuccess) { cudaGetLastError(); return 1; }   // a refused launch: the caller falls back and flags it
  return 0;
}

}  // namespace tc
}  // namespace mkv

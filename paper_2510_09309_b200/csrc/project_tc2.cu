// Mask-only projection, GEMM on pairs of CTAs (tcgen05 cta_group::2).
//
// With one CTA per tile the MMA reads the vocabulary tile from shared memory once per 128-row half of the masked
// rows, and together with the TMA writes that saturates the SM's shared-memory bandwidth before the tensor pipe is
// full.  Here two CTAs of a cluster share a tile of 256 rows x w vocabulary entries: each holds 128 of the packed
// rows and w/2 rows of the vocabulary tile, the leader's thread issues one M = 256 MMA for both, and each SM reads
// and writes about a third less shared memory per MMA cycle.  Per CTA an accumulator is 128 lanes x w <= 256 columns,
// so tensor memory holds two and a tile's epilogue runs under the next tile's products.
//   warp 0     TMA producer (both CTAs; all copies of a stage count on the leader's barrier)
//   warp 1     MMA issuer (leader only); commits arrive on the barriers of both CTAs
//   warps 2-5  epilogue (both CTAs): a thread owns an output row; a warp's lane 0 reports the drained accumulator to
//              the leader's barrier
// Every wait is bounded as in the other tensor-core kernels; both CTAs meet at a cluster barrier before they free
// tensor memory and leave, whatever happened before.
#include "project_tc.h"

#include "project_common.cuh"

namespace mkv {
namespace tc {

namespace {

constexpr int k2Threads = 192;
constexpr int k2Stages = 6;
constexpr int k2ABytes = 128 * 128;   // this CTA's 128 packed rows of a k block
constexpr int k2BarBytes = 256;

struct Bars2 {
  uint64_t* full;    // [k2Stages] operands of both CTAs landed (used in the leader)
  uint64_t* empty;   // [k2Stages] operands consumed (one in each CTA)
  uint64_t* tfull;   // [2] accumulator written (one in each CTA)
  uint64_t* tempty;  // [2] accumulator drained by the 8 epilogue warps of the pair (used in the leader)
};

__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
// Tile load into this CTA's shared memory whose bytes are counted on a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T with A = the 128 rows each CTA holds (M = 256) and B = the w/2 rows each holds.
__device__ __forceinline__ void umma_ss_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on `bar` in both CTAs of the pair once every MMA issued so far by this thread has completed: two plain
// commits, one on this CTA's barrier and one on the peer's copy of it (address from mapa); both track the same MMAs.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar, uint32_t peer_rank) {
  const uint32_t own = smem_u32(bar);
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(own) : "memory");
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(map_to_cta(own, peer_rank)) : "memory");
}

__global__ void __launch_bounds__(k2Threads, 1)
project_gemm_tc2(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w0,
                 const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w2, PPlan pl, int n_mask,
                 int vocab, int width, void* __restrict__ out, long long ld_out, int out_bf16, uint32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stage_bytes = k2ABytes + (pl.wmax / 2) * 128;
  uint64_t* bar0 = reinterpret_cast<uint64_t*>(base + k2Stages * stage_bytes);
  const Bars2 bars = {bar0, bar0 + k2Stages, bar0 + 2 * k2Stages, bar0 + 2 * k2Stages + 2};
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar0 + 2 * k2Stages + 4);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_cta_rank();                 // 0 = leader
  const int pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    prefetch_tmap(&map_a); prefetch_tmap(&map_w0); prefetch_tmap(&map_w1); prefetch_tmap(&map_w2);
    for (int s = 0; s < k2Stages; ++s) { mbar_init(bars.full + s, 1); mbar_init(bars.empty + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bars.tfull + b, 1); mbar_init(bars.tempty + b, 8); }
    *abort_flag = 0u;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
  tc_fence_before();
  cluster_sync_all();                                       // both CTAs' barriers exist before anything arrives on them
  tc_fence_after();
  pdl_wait();                                               // the packed rows come from the gather kernel
  const uint32_t tmem_base = *tmem_slot;

  const int m_blocks = (n_mask + kPBM - 1) / kPBM;
  const int k_blocks = (width + kPBK - 1) / kPBK;

  if (warp == 0) {
    if (lane == 0) {
      int it = 0;
      bool ok = true;
      for (int ti = 0; ok && ti < pl.n_t; ++ti) {
        int col0, w;
        project_tile(pl, pair, pairs, ti, &col0, &w);
        if (w == 0) continue;
        const CUtensorMap* map_w = w == pl.widths[0] ? &map_w0 : w == pl.widths[1] ? &map_w1 : &map_w2;
        for (int mb = 0; ok && mb < m_blocks; ++mb) {
          for (int kb = 0; kb < k_blocks; ++kb, ++it) {
            const int stage = it % k2Stages, use = it / k2Stages;
            if (!(ok = mbar_wait(bars.empty + stage, (use & 1) ^ 1, abort_flag, status, 0x310))) break;
            uint8_t* dst = base + stage * stage_bytes;
            if (rank == 0) mbar_expect_tx(bars.full + stage, (uint32_t)(2 * (k2ABytes + (w / 2) * 128)));
            const uint32_t full_leader = map_to_cta(smem_u32(bars.full + stage), 0);
            tma_load_2d_pair(dst, &map_a, full_leader, kb * kPBK, mb * kPBM + (int)rank * 128);
            tma_load_2d_pair(dst + k2ABytes, map_w, full_leader, kb * kPBK, col0 + (int)rank * (w / 2));
          }
        }
      }
      // Copies into this CTA's shared memory must have landed before it leaves.  Their bytes are counted in the
      // leader, so the peer cannot see them land; both CTAs instead wait (bounded) on the leader's last barriers
      // through the cluster barrier at the end: the leader drains here, the peer relies on that barrier.
      if (!ok && rank == 0)
        for (int i = max(0, it - k2Stages); i < it; ++i)
          for (uint32_t p = 0; p < (1u << 20) && !mbar_try_wait(bars.full + i % k2Stages, (i / k2Stages) & 1); ++p) __nanosleep(64);
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      const uint32_t lo_base = smem_desc_lo(smem_u32(base));
      int it = 0;
      uint32_t tile_i = 0;
      bool ok = true;
      for (int ti = 0; ok && ti < pl.n_t; ++ti) {
        int col0, w;
        project_tile(pl, pair, pairs, ti, &col0, &w);
        if (w == 0) continue;
        const uint32_t idesc = idesc_bf16_f32(256, (uint32_t)w);
        for (int mb = 0; ok && mb < m_blocks; ++mb, ++tile_i) {
          const uint32_t acc = tile_i & 1;
          if (!(ok = mbar_wait(bars.tempty + acc, ((tile_i >> 1) & 1) ^ 1, abort_flag, status, 0x311))) break;
          tc_fence_after();
          for (int kb = 0; kb < k_blocks; ++kb, ++it) {
            const int stage = it % k2Stages, use = it / k2Stages;
            if (!(ok = mbar_wait(bars.full + stage, use & 1, abort_flag, status, 0x312))) break;
            tc_fence_after();
            const uint32_t a_lo = lo_base + ((uint32_t)(stage * stage_bytes) >> 4);
            const uint32_t b_lo = a_lo + (k2ABytes >> 4);
#pragma unroll
            for (int kk = 0; kk < kPBK / 16; ++kk)
              umma_ss_pair(tmem_base + acc * 256, make_desc(a_lo + ((kk * 32) >> 4), kDescHiSw128),
                           make_desc(b_lo + ((kk * 32) >> 4), kDescHiSw128), idesc, (kb | kk) != 0);
            umma_commit_pair(bars.empty + stage, rank ^ 1u);
          }
          if (ok) umma_commit_pair(bars.tfull + acc, rank ^ 1u);
        }
      }
    }
  } else {
    const int lane_group = warp & 3;                        // the TMEM lanes this warp may read
    uint8_t* stg = base + k2Stages * stage_bytes + k2BarBytes + (warp - 2) * kPStageOutBytes;
    uint32_t tile_i = 0;
    bool ok = true;
    for (int ti = 0; ok && ti < pl.n_t; ++ti) {
      int tcol0, w;
      project_tile(pl, pair, pairs, ti, &tcol0, &w);
      if (w == 0) continue;
      const int chunks = (w + 31) / 32;                     // a last half chunk reads 16 stale columns and drops them
      const int col_end = min(vocab, tcol0 + w);
      for (int mb = 0; ok && mb < m_blocks; ++mb, ++tile_i) {
        const uint32_t acc = tile_i & 1;
        const int row0 = mb * kPBM + (int)rank * 128 + lane_group * 32;
        if (!(ok = mbar_wait(bars.tfull + acc, (tile_i >> 1) & 1, abort_flag, status, 0x313))) break;
        tc_fence_after();
        const uint32_t lane_addr = tmem_base + ((uint32_t)(lane_group * 32) << 16) + acc * 256;
        float va[32], vb[32];
        tmem_ld32(lane_addr, va);
        for (int c = 0; c < chunks; c += 2) {
          tmem_ld_wait();
          if (c + 1 < chunks) tmem_ld32(lane_addr + (c + 1) * 32, vb);
          project_store_chunk(va, stg, lane, row0, n_mask, tcol0 + c * 32, col_end, out, ld_out, out_bf16);
          if (c + 1 < chunks) {
            tmem_ld_wait();
            if (c + 2 < chunks) tmem_ld32(lane_addr + (c + 2) * 32, va);
            project_store_chunk(vb, stg, lane, row0, n_mask, tcol0 + (c + 1) * 32, col_end, out, ld_out, out_bf16);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(bars.tempty + acc), 0));
      }
    }
  }
  tc_fence_before();
  cluster_sync_all();                                       // nobody frees tensor memory or leaves while the peer works
  if (warp == 1) { tc_fence_after(); tmem_dealloc_pair(tmem_base, 512); }
}

size_t project2_smem_bytes(int wmax) {
  return (size_t)k2Stages * (k2ABytes + (wmax / 2) * 128) + 1024 + k2BarBytes + 4 * kPStageOutBytes;
}

}  // namespace

bool project_tc2_supported(const maskkv_ctx* ctx) {
  return ctx->encode_tiled != nullptr && (size_t)ctx->smem_optin >= project2_smem_bytes(256) && ctx->sm_count >= 2;
}

int launch_project_gemm_tc2(maskkv_ctx* ctx, const void* a_base, long long a_stride_bytes, int width, int n_mask, const void* w_vocab,
                            int vocab, long long w_row_stride, void* out, long long ld_out, int out_bf16, cudaStream_t st) {
  PPlan pl;
  const int pairs = make_project_plan(ctx->sm_count / 2, vocab, &pl);
  if (pairs == 0) return 1;
  CUtensorMap map_a, map_w[kPMaxWidths];
  if (!make_tmap_matrix(ctx->encode_tiled, &map_a, a_base, (uint64_t)width, (uint64_t)n_mask, (uint64_t)a_stride_bytes, 128)) return 1;
  for (int k = 0; k < kPMaxWidths; ++k)
    if (!make_tmap_matrix(ctx->encode_tiled, &map_w[k], w_vocab, (uint64_t)width, (uint64_t)vocab, (uint64_t)w_row_stride * 2,
                          (uint32_t)(pl.widths[k] / 2)))
      return 1;
  static bool attr_done[64] = {};
  if (ctx->device < 0 || ctx->device >= 64) return 1;
  if (!attr_done[ctx->device]) {
    if (cudaFuncSetAttribute(project_gemm_tc2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)project2_smem_bytes(256)) != cudaSuccess)
      return 1;
    attr_done[ctx->device] = true;
  }
  const cudaError_t e = launch_overlapped_cluster(project_gemm_tc2, dim3(2 * pairs), dim3(k2Threads), project2_smem_bytes(pl.wmax), st, 2u,
                                                  map_a, map_w[0], map_w[1], map_w[2], pl, n_mask, vocab, width, out, ld_out, out_bf16,
                                                  ctx->status_dev);
  if (e != cudaSuccess) return 1;
  ctx->tc_launches += 1;
  return 0;
}

}  // namespace tc
}  // namespace mkv

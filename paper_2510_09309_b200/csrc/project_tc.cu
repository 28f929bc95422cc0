// Mask-only projection (appendix, "Mask-only Projection") on the tensor cores:
//   logits[m, v] = sum_k hidden[positions[m], k] * w_vocab[v, k]        (bf16 x bf16 -> fp32)
//
// A gather kernel first packs the masked rows of the hidden state into a dense [n_mask][width] operand (a few MB that
// then stays in L2); the GEMM kernel is persistent, one CTA per SM, and streams the vocabulary matrix exactly once:
//   warp 0     TMA producer: per 64-wide k block one [256 rows x 64] box of the packed rows and one [tile width x 64] box of w_vocab
//   warp 1     one thread issues tcgen05.mma (M = 128 twice, N = tile width, K = 16 x 4 per block) into two TMEM accumulators
//   warps 2-9  epilogue: a thread owns an output row, reads it from TMEM 32 columns at a time and stores it
// The vocabulary is shared out as project_common.cuh describes; a CTA runs all row
// blocks (256 masked rows each) of a tile before it moves on, so a vocabulary tile comes from DRAM once.  Both
// accumulators can take all of tensor memory, so a tile's epilogue is not overlapped with the next tile's products;
// it is about 2 % of a tile's time at width 4096.
#include "project_tc.h"

#include "project_common.cuh"

namespace mkv {
namespace tc {

namespace {

constexpr int kPThreads = 320;        // TMA warp, MMA warp, 8 epilogue warps
constexpr int kPStages = 3;
constexpr int kPABytes = kPBM * 128;  // packed-rows operand per stage
constexpr int kPBarBytes = 128;       // mbarriers, tensor-memory base, abort flag
struct PBars {
  uint64_t* full;    // [kPStages] operands landed
  uint64_t* empty;   // [kPStages] operands consumed
  uint64_t* tfull;   // accumulators written
  uint64_t* tempty;  // accumulators drained (256 epilogue threads)
};

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
               : "memory");
}

// One warp per masked position: copies its hidden row (16-byte pieces) into the packed operand; a position outside
// the sequence raises the bounds flag and leaves a zero row.
__global__ void __launch_bounds__(256)
project_gather_kernel(const unsigned char* __restrict__ hidden, long long row_stride_bytes, long long n_tokens,
                      const int32_t* __restrict__ positions, int n_mask, int row_bytes, unsigned char* __restrict__ packed,
                      uint32_t* __restrict__ status) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  for (int m = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; m < n_mask; m += warps) {
    const long long p = positions[m];
    const bool ok = p >= 0 && p < n_tokens;
    if (!ok && lane == 0) atomicOr(status, (uint32_t)MASKKV_FLAG_BOUNDS);
    const uint4* src = reinterpret_cast<const uint4*>(hidden + (ok ? p : 0) * row_stride_bytes);
    uint4* dst = reinterpret_cast<uint4*>(packed + (long long)m * row_bytes);
    for (int e = lane; e < row_bytes / 16; e += 32) dst[e] = ok ? __ldg(src + e) : make_uint4(0u, 0u, 0u, 0u);
  }
}

// out: fp32 or bf16 rows of ld_out elements.  Tiles are numbered (vocabulary tile, row block) with the row block
// fastest, so the CTAs that share a vocabulary tile run at the same time and it is fetched from DRAM once.
__global__ void __launch_bounds__(kPThreads, 1)
project_gemm_tc(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w0,
                const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w2, PPlan pl, int n_mask,
                int vocab, int width, void* __restrict__ out, long long ld_out, int out_bf16, uint32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stage_bytes = kPABytes + pl.wmax * 128;
  uint64_t* bar0 = reinterpret_cast<uint64_t*>(base + kPStages * stage_bytes);
  const PBars bars = {bar0, bar0 + kPStages, bar0 + 2 * kPStages, bar0 + 2 * kPStages + 1};
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar0 + 2 * kPStages + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    prefetch_tmap(&map_a); prefetch_tmap(&map_w0); prefetch_tmap(&map_w1); prefetch_tmap(&map_w2);
    for (int s = 0; s < kPStages; ++s) { mbar_init(bars.full + s, 1); mbar_init(bars.empty + s, 1); }
    mbar_init(bars.tfull, 1); mbar_init(bars.tempty, 256);
    *abort_flag = 0u;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();                                               // the packed rows come from the gather kernel
  const uint32_t tmem_base = *tmem_slot;

  const int m_blocks = (n_mask + kPBM - 1) / kPBM;
  const int k_blocks = (width + kPBK - 1) / kPBK;           // a ragged last block reads zeros past the row's end

  if (warp == 0) {
    if (lane == 0) {
      int it = 0;
      bool ok = true;
      for (int ti = 0; ok && ti < pl.n_t; ++ti) {
        int col0, w;
        project_tile(pl, blockIdx.x, gridDim.x, ti, &col0, &w);
        if (w == 0) continue;
        const CUtensorMap* map_w = w == pl.widths[0] ? &map_w0 : w == pl.widths[1] ? &map_w1 : &map_w2;
        for (int mb = 0; ok && mb < m_blocks; ++mb) {
          for (int kb = 0; kb < k_blocks; ++kb, ++it) {
            const int stage = it % kPStages, use = it / kPStages;
            if (!(ok = mbar_wait(bars.empty + stage, (use & 1) ^ 1, abort_flag, status, 0x300))) break;
            uint8_t* dst = base + stage * stage_bytes;
            mbar_expect_tx(bars.full + stage, (uint32_t)(kPABytes + w * 128));
            tma_load_2d(dst, &map_a, bars.full + stage, kb * kPBK, mb * kPBM);
            tma_load_2d(dst + kPABytes, map_w, bars.full + stage, kb * kPBK, col0);
          }
        }
      }
      if (!ok)                                              // copies already issued must land before the block leaves
        for (int i = max(0, it - kPStages); i < it; ++i)
          for (uint32_t p = 0; p < (1u << 20) && !mbar_try_wait(bars.full + i % kPStages, (i / kPStages) & 1); ++p) __nanosleep(64);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t lo_base = smem_desc_lo(smem_u32(base));
      int it = 0;
      uint32_t tile_i = 0;
      bool ok = true;
      for (int ti = 0; ok && ti < pl.n_t; ++ti) {
        int col0, w;
        project_tile(pl, blockIdx.x, gridDim.x, ti, &col0, &w);
        if (w == 0) continue;
        const uint32_t idesc = idesc_bf16_f32(128, (uint32_t)w);
        for (int mb = 0; ok && mb < m_blocks; ++mb, ++tile_i) {
          const int halves = n_mask - mb * kPBM > 128 ? 2 : 1;
          if (!(ok = mbar_wait(bars.tempty, (tile_i & 1) ^ 1, abort_flag, status, 0x301))) break;
          tc_fence_after();
          for (int kb = 0; kb < k_blocks; ++kb, ++it) {
            const int stage = it % kPStages, use = it / kPStages;
            if (!(ok = mbar_wait(bars.full + stage, use & 1, abort_flag, status, 0x302))) break;
            tc_fence_after();
            const uint32_t a_lo = lo_base + ((uint32_t)(stage * stage_bytes) >> 4);
            const uint32_t b_lo = a_lo + (kPABytes >> 4);
            for (int a = 0; a < halves; ++a) {
#pragma unroll
              for (int kk = 0; kk < kPBK / 16; ++kk)
                umma_ss(tmem_base + a * 256, make_desc(a_lo + ((a * 128 * 128 + kk * 32) >> 4), kDescHiSw128),
                        make_desc(b_lo + ((kk * 32) >> 4), kDescHiSw128), idesc, (kb | kk) != 0);
            }
            umma_commit(bars.empty + stage);
          }
          if (ok) umma_commit(bars.tfull);
        }
      }
    }
  } else {
    const int a = (warp - 2) >> 2;
    const int lane_group = warp & 3;                        // the TMEM lanes this warp may read
    const uint32_t lane_addr = tmem_base + ((uint32_t)(lane_group * 32) << 16) + a * 256;
    uint8_t* stg = base + kPStages * stage_bytes + kPBarBytes + (warp - 2) * kPStageOutBytes;
    uint32_t tile_i = 0;
    bool ok = true;
    for (int ti = 0; ok && ti < pl.n_t; ++ti) {
     int tcol0, w;
     project_tile(pl, blockIdx.x, gridDim.x, ti, &tcol0, &w);
     if (w == 0) continue;
     const int chunks = (w + 31) / 32;                       // a last half chunk reads 16 stale columns and drops them
     const int col_end = min(vocab, tcol0 + w);
     for (int mb = 0; ok && mb < m_blocks; ++mb, ++tile_i) {
      const bool half_used = n_mask - mb * kPBM > a * 128;  // warp-uniform: the MMA warp skips an empty second half
      if (!(ok = mbar_wait(bars.tfull, tile_i & 1, abort_flag, status, 0x303))) break;
      tc_fence_after();
      if (half_used) {
        float va[32], vb[32];
        const int row0 = mb * kPBM + a * 128 + lane_group * 32;
        auto store = [&](const float* v, int cc) {
          project_store_chunk(v, stg, lane, row0, n_mask, tcol0 + cc * 32, col_end, out, ld_out, out_bf16);
        };
        tmem_ld32(lane_addr, va);
        for (int c = 0; c < chunks; c += 2) {
          tmem_ld_wait();
          if (c + 1 < chunks) tmem_ld32(lane_addr + (c + 1) * 32, vb);
          store(va, c);
          if (c + 1 < chunks) {
            tmem_ld_wait();
            if (c + 2 < chunks) tmem_ld32(lane_addr + (c + 2) * 32, va);
            store(vb, c + 1);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bars.tempty);
     }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

size_t project_smem_bytes(int wmax) { return (size_t)kPStages * (kPABytes + wmax * 128) + 1024 + kPBarBytes + 8 * kPStageOutBytes; }

}  // namespace

bool project_tc_supported(const maskkv_ctx* ctx) {
  return ctx->encode_tiled != nullptr && (size_t)ctx->smem_optin >= project_smem_bytes(256);
}

int launch_project_tc(maskkv_ctx* ctx, const void* hidden, long long n_tokens, int width, long long hidden_row_stride,
                      const int32_t* positions, int n_mask, const void* w_vocab, int vocab, long long w_row_stride, void* out,
                      long long ld_out, int out_bf16, void* packed, cudaStream_t st, int* launches) {
  *launches = 0;
  const void* a_base = hidden;
  long long a_stride = hidden_row_stride * 2;
  PPlan pl;
  const int grid = make_project_plan(ctx->sm_count, vocab, &pl);
  if (grid == 0) return 1;
  CUtensorMap map_a, map_w[kPMaxWidths];
  if (positions != nullptr) { a_base = packed; a_stride = (long long)width * 2; }
  if (!make_tmap_matrix(ctx->encode_tiled, &map_a, a_base, (uint64_t)width, (uint64_t)n_mask, (uint64_t)a_stride, kPBM)) return 1;
  for (int k = 0; k < kPMaxWidths; ++k)
    if (!make_tmap_matrix(ctx->encode_tiled, &map_w[k], w_vocab, (uint64_t)width, (uint64_t)vocab, (uint64_t)w_row_stride * 2,
                          (uint32_t)pl.widths[k]))
      return 1;
  const size_t smem = project_smem_bytes(pl.wmax);
  static bool attr_done[64] = {};
  if (ctx->device < 0 || ctx->device >= 64) return 1;
  if (!attr_done[ctx->device]) {
    if (cudaFuncSetAttribute(project_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)project_smem_bytes(256)) != cudaSuccess)
      return 1;
    attr_done[ctx->device] = true;
  }
  if (positions != nullptr) {
    const int blocks = (n_mask + 7) / 8;
    project_gather_kernel<<<blocks < 1 ? 1 : blocks, 256, 0, st>>>(static_cast<const unsigned char*>(hidden), hidden_row_stride * 2,
                                                                   n_tokens, positions, n_mask, width * 2,
                                                                   static_cast<unsigned char*>(packed), ctx->status_dev);
    ++*launches;
  }
  // More than 128 masked rows: a pair of CTAs per tile (project_tc2.cu); otherwise the second CTA would have no rows.
  if (n_mask > 128 && !(ctx->kernel_choice & 1u) && project_tc2_supported(ctx)) {
    if (launch_project_gemm_tc2(ctx, a_base, a_stride, width, n_mask, w_vocab, vocab, w_row_stride, out, ld_out, out_bf16, st) != 0)
      return *launches == 0 ? 1 : 2;
    ++*launches;
    return 0;
  }
  launch_overlapped(project_gemm_tc, dim3(grid), dim3(kPThreads), smem, st, map_a, map_w[0], map_w[1], map_w[2], pl, n_mask, vocab,
                    width, out, ld_out, out_bf16, ctx->status_dev);
  ++*launches;
  ctx->tc_launches += 1;
  return 0;
}

}  // namespace tc
}  // namespace mkv

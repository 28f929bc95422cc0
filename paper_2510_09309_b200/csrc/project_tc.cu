// Mask-only projection (appendix, "Mask-only Projection") on the tensor cores:
//   logits[m, v] = sum_k hidden[positions[m], k] * w_vocab[v, k]        (bf16 x bf16 -> fp32)
//
// A gather kernel first packs the masked rows of the hidden state into a dense [n_mask][width] operand (a few MB that
// then stays in L2); the GEMM kernel is persistent, one CTA per SM, and streams the vocabulary matrix exactly once:
//   warp 0     TMA producer: per 64-wide k block one [256 rows x 64] box of the packed rows and one [BN x 64] box of w_vocab
//   warp 1     one thread issues tcgen05.mma (M = 128 twice, N = BN, K = 16 x 4 per block) into two TMEM accumulators
//   warps 2-9  epilogue: a thread owns an output row, reads it from TMEM 32 columns at a time and stores it
// An output tile is 256 rows x BN vocabulary entries; BN (128...256) is chosen on the host so that the tiles fill
// the last wave of CTAs as evenly as possible.  Both accumulators take all of tensor memory at BN = 256, so the
// epilogue of a tile is not overlapped with the next tile's products; it is about 2 % of a tile's time at width 4096.
#include "project_tc.h"

#include "tc_common.cuh"

namespace mkv {
namespace tc {

namespace {

constexpr int kPThreads = 320;        // TMA warp, MMA warp, 8 epilogue warps
constexpr int kPStages = 3;
constexpr int kPBM = 256;             // output rows per tile (two accumulators of 128)
constexpr int kPBK = 64;              // bf16 per k block = one 128-byte swizzled box row
constexpr int kPABytes = kPBM * 128;  // packed-rows operand per stage

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

__device__ __forceinline__ void st_stream4(float* p, float a, float b, float c, float d) {
  asm volatile("st.global.cs.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void st_stream4u(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
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
project_gemm_tc(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, int n_mask, int vocab,
                int width, int BN, void* __restrict__ out, long long ld_out, int out_bf16, uint32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stage_bytes = kPABytes + BN * 128;
  uint64_t* bar0 = reinterpret_cast<uint64_t*>(base + kPStages * stage_bytes);
  const PBars bars = {bar0, bar0 + kPStages, bar0 + 2 * kPStages, bar0 + 2 * kPStages + 1};
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar0 + 2 * kPStages + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    prefetch_tmap(&map_a); prefetch_tmap(&map_w);
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
  const int n_tiles = (vocab + BN - 1) / BN;
  const long long tiles = (long long)m_blocks * n_tiles;
  const int k_blocks = (width + kPBK - 1) / kPBK;           // a ragged last block reads zeros past the row's end

  if (warp == 0) {
    if (lane == 0) {
      int it = 0;
      bool ok = true;
      for (long long t = blockIdx.x; ok && t < tiles; t += gridDim.x) {
        const int mb = (int)(t % m_blocks), nt = (int)(t / m_blocks);
        for (int kb = 0; kb < k_blocks; ++kb, ++it) {
          const int stage = it % kPStages, use = it / kPStages;
          if (!(ok = mbar_wait(bars.empty + stage, (use & 1) ^ 1, abort_flag, status, 0x300))) break;
          uint8_t* dst = base + stage * stage_bytes;
          mbar_expect_tx(bars.full + stage, (uint32_t)stage_bytes);
          tma_load_2d(dst, &map_a, bars.full + stage, kb * kPBK, mb * kPBM);
          tma_load_2d(dst + kPABytes, &map_w, bars.full + stage, kb * kPBK, nt * BN);
        }
      }
      if (!ok)                                              // copies already issued must land before the block leaves
        for (int i = max(0, it - kPStages); i < it; ++i)
          for (uint32_t p = 0; p < (1u << 20) && !mbar_try_wait(bars.full + i % kPStages, (i / kPStages) & 1); ++p) __nanosleep(64);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(128, (uint32_t)BN);
      const uint32_t lo_base = smem_desc_lo(smem_u32(base));
      int it = 0;
      uint32_t tile_i = 0;
      bool ok = true;
      for (long long t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++tile_i) {
        const int mb = (int)(t % m_blocks);
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
  } else {
    const int a = (warp - 2) >> 2;
    const int lane_group = warp & 3;                        // the TMEM lanes this warp may read
    const uint32_t lane_addr = tmem_base + ((uint32_t)(lane_group * 32) << 16) + a * 256;
    const int chunks = BN / 32;
    uint32_t tile_i = 0;
    bool ok = true;
    for (long long t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++tile_i) {
      const int mb = (int)(t % m_blocks), nt = (int)(t / m_blocks);
      const int row = mb * kPBM + a * 128 + lane_group * 32 + lane;
      const bool half_used = n_mask - mb * kPBM > a * 128;  // warp-uniform: the MMA warp skips an empty second half
      if (!(ok = mbar_wait(bars.tfull, tile_i & 1, abort_flag, status, 0x303))) break;
      tc_fence_after();
      if (half_used) {
        float va[32], vb[32];
        tmem_ld32(lane_addr, va);
        for (int c = 0; c < chunks; c += 2) {
          tmem_ld_wait();
          if (c + 1 < chunks) tmem_ld32(lane_addr + (c + 1) * 32, vb);
          auto store = [&](const float* v, int cc) {
            const int col = nt * BN + cc * 32;
            if (row >= n_mask || col >= vocab) return;
            if (col + 32 <= vocab) {
              if (out_bf16) {
                uint4* p = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(out) + row * ld_out + col);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                  st_stream4u(p + i, bf16x2(v[8 * i], v[8 * i + 1]), bf16x2(v[8 * i + 2], v[8 * i + 3]),
                              bf16x2(v[8 * i + 4], v[8 * i + 5]), bf16x2(v[8 * i + 6], v[8 * i + 7]));
              } else {
                float* p = static_cast<float*>(out) + row * ld_out + col;
#pragma unroll
                for (int i = 0; i < 8; ++i) st_stream4(p + 4 * i, v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
              }
            } else {                                          // ragged end of the vocabulary
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                if (col + i >= vocab) continue;
                if (out_bf16) static_cast<__nv_bfloat16*>(out)[row * ld_out + col + i] = __float2bfloat16_rn(v[i]);
                else static_cast<float*>(out)[row * ld_out + col + i] = v[i];
              }
            }
          };
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
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

// [rows][width] bf16 matrix with a byte row stride, viewed as (width, rows); box = 64 x box_rows, 128-byte swizzle,
// zeros outside the matrix.
bool make_tmap_matrix(void* encode_fn, CUtensorMap* map, const void* base_ptr, uint64_t width, uint64_t rows,
                      uint64_t row_stride_bytes, uint32_t box_rows) {
  if (encode_fn == nullptr || base_ptr == nullptr || rows == 0 || width == 0) return false;
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  const cuuint64_t dims[2] = {width, rows};
  const cuuint64_t strides[1] = {row_stride_bytes};
  const cuuint32_t box[2] = {(cuuint32_t)kPBK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return reinterpret_cast<EncodeFn>(encode_fn)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base_ptr), dims, strides,
                                               box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t project_smem_bytes(int BN) { return (size_t)kPStages * (kPABytes + BN * 128) + 1024 + 128; }

}  // namespace

int project_tile_width(int sm_count, int n_mask, int vocab) {
  const long long m_blocks = (n_mask + kPBM - 1) / kPBM;
  int best = 256;
  long long best_cost = -1;
  for (int bn = 256; bn >= 128; bn -= 32) {
    const long long tiles = m_blocks * ((vocab + bn - 1) / bn);
    const long long cost = (tiles + sm_count - 1) / sm_count * bn;   // waves x time of a tile
    if (best_cost < 0 || cost < best_cost) { best = bn; best_cost = cost; }
  }
  return best;
}

bool project_tc_supported(const maskkv_ctx* ctx) {
  return ctx->encode_tiled != nullptr && (size_t)ctx->smem_optin >= project_smem_bytes(256);
}

int launch_project_tc(maskkv_ctx* ctx, const void* hidden, long long n_tokens, int width, long long hidden_row_stride,
                      const int32_t* positions, int n_mask, const void* w_vocab, int vocab, long long w_row_stride, void* out,
                      long long ld_out, int out_bf16, void* packed, cudaStream_t st, int* launches) {
  *launches = 0;
  const void* a_base = hidden;
  long long a_stride = hidden_row_stride * 2;
  const int BN = project_tile_width(ctx->sm_count, n_mask, vocab);
  CUtensorMap map_a, map_w;
  if (positions != nullptr) { a_base = packed; a_stride = (long long)width * 2; }
  if (!make_tmap_matrix(ctx->encode_tiled, &map_a, a_base, (uint64_t)width, (uint64_t)n_mask, (uint64_t)a_stride, kPBM) ||
      !make_tmap_matrix(ctx->encode_tiled, &map_w, w_vocab, (uint64_t)width, (uint64_t)vocab, (uint64_t)w_row_stride * 2, (uint32_t)BN))
    return 1;
  const size_t smem = project_smem_bytes(BN);
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
  const long long tiles = (long long)((n_mask + kPBM - 1) / kPBM) * ((vocab + BN - 1) / BN);
  const int grid = (int)(tiles < ctx->sm_count ? tiles : ctx->sm_count);
  launch_overlapped(project_gemm_tc, dim3(grid), dim3(kPThreads), smem, st, map_a, map_w, n_mask, vocab, width, BN, out, ld_out,
                    out_bf16, ctx->status_dev);
  ++*launches;
  ctx->tc_launches += 1;
  return 0;
}

}  // namespace tc
}  // namespace mkv

// Mask-only projection (appendix, "Mask-only Projection") on the tensor cores:
//   logits[m, v] = sum_k hidden[positions[m], k] * w_vocab[v, k]        (bf16 x bf16 -> fp32)
//
// A gather kernel first packs the masked rows of the hidden state into a dense [n_mask][width] operand (a few MB that
// then stays in L2); the GEMM kernel is persistent, one CTA per SM, and streams the vocabulary matrix exactly once:
//   warp 0     TMA producer: per 64-wide k block one [256 rows x 64] box of the packed rows and one [tile width x 64] box of w_vocab
//   warp 1     one thread issues tcgen05.mma (M = 128 twice, N = tile width, K = 16 x 4 per block) into two TMEM accumulators
//   warps 2-9  epilogue: a thread owns an output row, reads it from TMEM 32 columns at a time and stores it
// The vocabulary is cut into units of 16 entries (the granularity of the MMA's N); CTA c of G owns the contiguous
// units [c*U/G, (c+1)*U/G) and cuts them into the same number of tiles as every other CTA, so all CTAs carry the same
// load to within one unit and tile widths take at most three values (one tensor map each).  A CTA runs all row
// blocks (256 masked rows each) of a tile before it moves on, so a vocabulary tile comes from DRAM once.  Both
// accumulators can take all of tensor memory, so a tile's epilogue is not overlapped with the next tile's products;
// it is about 2 % of a tile's time at width 4096.
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
constexpr int kPBarBytes = 128;       // mbarriers, tensor-memory base, abort flag
constexpr int kPStageOutBytes = 4096; // per epilogue warp: 32 rows x 128 bytes on their way out

constexpr int kPMaxWidths = 3;

// How the vocabulary is shared out (see the top of the file).  widths[] are the tile widths that occur, in entries.
struct PPlan {
  int units;                 // ceil(vocab / 16)
  int n_t;                   // tiles per CTA
  int widths[kPMaxWidths];   // ascending; unused entries repeat the last one
  int wmax;
};
// Tile ti of this CTA: first vocabulary entry and width (0 = no such tile).
__host__ __device__ __forceinline__ void project_tile(const PPlan& pl, int cta, int G, int ti, int* col0, int* w) {
  const long long u0 = (long long)cta * pl.units / G, u1 = (long long)(cta + 1) * pl.units / G;
  const long long share = u1 - u0;
  const long long t0 = u0 + share * ti / pl.n_t, t1 = u0 + share * (ti + 1) / pl.n_t;
  *col0 = (int)(t0 * 16);
  *w = (int)((t1 - t0) * 16);
}

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
        // A thread holds 32 consecutive logits of its own row; stored like that a warp's store instruction would touch
        // 32 different lines.  The chunk goes through a 4 KB staging block instead (16-byte pieces, XOR-swizzled so
        // that neither side has bank conflicts) and leaves as whole 128-byte (fp32) or 64-byte (bf16) row pieces.
        float va[32], vb[32];
        const int row0 = mb * kPBM + a * 128 + lane_group * 32;
        auto store = [&](const float* v, int cc) {
          const int col0 = tcol0 + cc * 32;
          if (col0 >= col_end) return;                          // warp-uniform
          if (out_bf16) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              *reinterpret_cast<uint4*>(stg + lane * 64 + 16 * (j ^ ((lane >> 1) & 3))) =
                  make_uint4(bf16x2(v[8 * j], v[8 * j + 1]), bf16x2(v[8 * j + 2], v[8 * j + 3]), bf16x2(v[8 * j + 4], v[8 * j + 5]),
                             bf16x2(v[8 * j + 6], v[8 * j + 7]));
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int rl = 8 * i + (lane >> 2), piece = lane & 3;
              const uint4 x = *reinterpret_cast<const uint4*>(stg + rl * 64 + 16 * (piece ^ ((rl >> 1) & 3)));
              const int row = row0 + rl, col = col0 + piece * 8;
              if (row >= n_mask || col >= col_end) continue;
              __nv_bfloat16* p = static_cast<__nv_bfloat16*>(out) + row * ld_out + col;
              if (col + 8 <= col_end) st_stream4u(p, x.x, x.y, x.z, x.w);
              else {
                const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&x);
                for (int k = 0; k < 8 && col + k < col_end; ++k) p[k] = e[k];
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              *reinterpret_cast<float4*>(stg + lane * 128 + 16 * (j ^ (lane & 7))) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int rl = 4 * i + (lane >> 3), piece = lane & 7;
              const float4 x = *reinterpret_cast<const float4*>(stg + rl * 128 + 16 * (piece ^ (rl & 7)));
              const int row = row0 + rl, col = col0 + piece * 4;
              if (row >= n_mask || col >= col_end) continue;
              float* p = static_cast<float*>(out) + row * ld_out + col;
              if (col + 4 <= col_end) st_stream4(p, x.x, x.y, x.z, x.w);
              else {
                const float e[4] = {x.x, x.y, x.z, x.w};
                for (int k = 0; k < 4 && col + k < col_end; ++k) p[k] = e[k];
              }
            }
          }
          __syncwarp();                                       // the block is free for the next chunk
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

size_t project_smem_bytes(int wmax) { return (size_t)kPStages * (kPABytes + wmax * 128) + 1024 + kPBarBytes + 8 * kPStageOutBytes; }

// Grid and plan for a vocabulary of `vocab` entries on `sm_count` SMs: every CTA gets at least four units (64 entries)
// when there are that many, and the same number of tiles, each at most 256 entries wide.
int make_plan(int sm_count, int vocab, PPlan* pl) {
  pl->units = (vocab + 15) / 16;
  int G = (pl->units + 3) / 4;
  if (G > sm_count) G = sm_count;
  if (G < 1) G = 1;
  const int max_share = (pl->units + G - 1) / G;
  pl->n_t = (max_share + 15) / 16;
  int n = 0;
  for (int c = 0; c < G; ++c)
    for (int ti = 0; ti < pl->n_t; ++ti) {
      int col0, w;
      project_tile(*pl, c, G, ti, &col0, &w);
      if (w == 0) continue;
      bool seen = false;
      for (int k = 0; k < n; ++k) seen = seen || pl->widths[k] == w;
      if (seen) continue;
      if (n == kPMaxWidths) return 0;                        // cannot happen: shares differ by one unit at most
      pl->widths[n++] = w;
    }
  if (n == 0) return 0;
  for (int k = n; k < kPMaxWidths; ++k) pl->widths[k] = pl->widths[n - 1];
  pl->wmax = 0;
  for (int k = 0; k < kPMaxWidths; ++k) pl->wmax = pl->widths[k] > pl->wmax ? pl->widths[k] : pl->wmax;
  return G;
}

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
  const int grid = make_plan(ctx->sm_count, vocab, &pl);
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
  launch_overlapped(project_gemm_tc, dim3(grid), dim3(kPThreads), smem, st, map_a, map_w[0], map_w[1], map_w[2], pl, n_mask, vocab,
                    width, out, ld_out, out_bf16, ctx->status_dev);
  ++*launches;
  ctx->tc_launches += 1;
  return 0;
}

}  // namespace tc
}  // namespace mkv

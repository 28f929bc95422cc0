// Pieces shared by the two GEMM kernels of the mask-only projection (project_tc.cu: one CTA per tile;
// project_tc2.cu: a pair of CTAs per tile): how the vocabulary is shared out, and the way a chunk of logits leaves
// the registers.
#pragma once

#include "tc_common.cuh"

namespace mkv {
namespace tc {

constexpr int kPBM = 256;             // output rows per tile
constexpr int kPBK = 64;              // bf16 per k block = one 128-byte swizzled box row
constexpr int kPStageOutBytes = 4096; // per epilogue warp: 32 rows x 128 bytes on their way out
constexpr int kPMaxWidths = 3;

// The vocabulary is cut into units of 16 entries (the granularity of the MMA's N).  Worker c of G (a CTA, or a pair
// of CTAs) owns the contiguous units [c*U/G, (c+1)*U/G) and cuts them into the same number of tiles as every other
// worker, so all carry the same load to within one unit and tile widths take at most three values (one tensor map
// each).  widths[] are the tile widths that occur, in entries.
struct PPlan {
  int units;                 // ceil(vocab / 16)
  int n_t;                   // tiles per worker
  int widths[kPMaxWidths];   // unused entries repeat the last one
  int wmax;
};
// Tile ti of worker c: first vocabulary entry and width (0 = no such tile).
__host__ __device__ __forceinline__ void project_tile(const PPlan& pl, int c, int G, int ti, int* col0, int* w) {
  const long long u0 = (long long)c * pl.units / G, u1 = (long long)(c + 1) * pl.units / G;
  const long long share = u1 - u0;
  const long long t0 = u0 + share * ti / pl.n_t, t1 = u0 + share * (ti + 1) / pl.n_t;
  *col0 = (int)(t0 * 16);
  *w = (int)((t1 - t0) * 16);
}

// Number of workers (at most max_workers; each gets at least four units when there are that many) and the plan.
// 0 = no plan (cannot happen for vocab > 0: shares differ by one unit at most, so at most three widths occur).
inline int make_project_plan(int max_workers, int vocab, PPlan* pl) {
  pl->units = (vocab + 15) / 16;
  int G = (pl->units + 3) / 4;
  if (G > max_workers) G = max_workers;
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
      if (n == kPMaxWidths) return 0;
      pl->widths[n++] = w;
    }
  if (n == 0) return 0;
  for (int k = n; k < kPMaxWidths; ++k) pl->widths[k] = pl->widths[n - 1];
  pl->wmax = 0;
  for (int k = 0; k < kPMaxWidths; ++k) pl->wmax = pl->widths[k] > pl->wmax ? pl->widths[k] : pl->wmax;
  return G;
}

// [rows][width] bf16 matrix with a byte row stride, viewed as (width, rows); box = 64 x box_rows, 128-byte swizzle,
// zeros outside the matrix.
inline bool make_tmap_matrix(void* encode_fn, CUtensorMap* map, const void* base_ptr, uint64_t width, uint64_t rows,
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

// A warp's 32 rows x 32 logits (lane = row row0 + lane, v = its 32 consecutive logits from column col0) go out.
// Stored straight from the registers a warp's store instruction would touch 32 different lines; the chunk goes
// through the warp's 4 KB staging block instead (16-byte pieces, XOR-swizzled so that neither side has bank
// conflicts) and leaves as whole 128-byte (fp32) or 64-byte (bf16) row pieces.  Entries from col_end on and rows from
// n_rows on are dropped.  Called by all 32 lanes.
__device__ __forceinline__ void project_store_chunk(const float* v, uint8_t* stg, int lane, int row0, int n_rows, int col0, int col_end,
                                                    void* out, long long ld_out, int out_bf16) {
  if (col0 >= col_end) return;                              // warp-uniform
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
      if (row >= n_rows || col >= col_end) continue;
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
      if (row >= n_rows || col >= col_end) continue;
      float* p = static_cast<float*>(out) + row * ld_out + col;
      if (col + 4 <= col_end) st_stream4(p, x.x, x.y, x.z, x.w);
      else {
        const float e[4] = {x.x, x.y, x.z, x.w};
        for (int k = 0; k < 4 && col + k < col_end; ++k) p[k] = e[k];
      }
    }
  }
  __syncwarp();                                             // the block is free for the next chunk
}

}  // namespace tc
}  // namespace mkv

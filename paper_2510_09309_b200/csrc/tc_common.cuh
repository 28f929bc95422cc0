// Blackwell (sm_100a) building blocks used by the tensor-core kernels: mbarriers with bounded
// waits, TMA tile loads, tensor-memory allocation, tcgen05 MMA issue / commit / load, and the
// shared-memory matrix descriptors for 128-byte-swizzled K-major operand tiles.
//
// Conventions
//   * Operand tiles are [rows][64] bf16 boxes (128 bytes per row) written by TMA with the 128-byte
//     swizzle; a head_dim of 128 is two such boxes.  Tile bases are 1024-byte aligned, groups of 8
//     rows are 1024 bytes apart, and the k-th 16-element slice of a box starts 32*k bytes in.
//   * Every wait on an mbarrier gives up after a bounded time (about one second), raises
//     MASKKV_FLAG_TIMEOUT in the status word and makes the whole block leave its loops; nothing
//     in these kernels can spin forever.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace mkv {
namespace tc {

constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // a wait gives up after about a second

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Block-wide abort protocol: `abort_flag` lives in shared memory; once set every role stops waiting.
// Returns false when the wait was abandoned (by this thread's limit or by another thread's).
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint32_t where) {
  // No sleeping between polls: try_wait already blocks for a short, hardware-chosen time, and the kernels that use
  // this are latency chains.  The limit is wall time (kWaitLimitNs), checked every 256 polls.
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) break;
    }
  }
  *abort_flag = 1u;
  atomicOr(status, (uint32_t)MASKKV_FLAG_TIMEOUT);
  atomicExch(status + 1, where);
  return false;
}

// ---------------------------------------------------------------- TMA (tile mode, no cluster features)
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// Brings the tile into L2 only (no shared memory, no barrier): hides the DRAM latency of a later tma_load_3d.
__device__ __forceinline__ void tma_prefetch_l2_3d(const CUtensorMap* map, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(map), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---------------------------------------------------------------- tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp gets lane (base lane + t), columns [col, col+32).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t* u = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
        "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]),
        "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]),
        "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------- MMA
// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4)     // start address, 16-byte units
         | ((uint64_t)1 << 16)                   // leading byte offset (unused for swizzled K-major)
         | ((uint64_t)(1024 >> 4) << 32)         // stride byte offset between 8-row groups
         | ((uint64_t)1 << 46)                   // descriptor version of this architecture
         | ((uint64_t)2 << 61);                  // 128-byte swizzle
}
// The same descriptor split in two words so that the issuing thread only adds a constant per MMA: the high word
// never changes and the low word is (address >> 4) | (1 << 16); advancing the operand by `bytes` adds bytes >> 4
// (shared-memory addresses stay below 256 KB, so the sum never leaves the 14-bit address field).
constexpr uint32_t kDescHiSw128 = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t saddr) { return ((saddr & 0x3ffffu) >> 4) | (1u << 16); }
__device__ __forceinline__ uint64_t make_desc(uint32_t lo, uint32_t hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}
// Instruction descriptor of kind::f16: bf16 x bf16 -> fp32, both operands K-major, tile m x n.
__host__ __device__ __forceinline__ uint32_t idesc_bf16_f32(uint32_t m, uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((m >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]^T, issued by one thread.
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on `bar` once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Packed fp32 pairs (two floats in one 64-bit register): one issue slot does the work of two.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// 2^x on the FMA pipes, for the share of the exponentials that the special-function unit (16 results per clock per SM)
// has no time for.  x = v*c + K with K an INTEGER known beforehand (the caller folds every fractional constant into a
// later multiplication): adding the magic number 1.5 * 2^23 + K inside the multiply-add rounds v*c to the nearest
// integer n and leaves n + K in the low mantissa bits; f = v*c - n lies in [-0.5, 0.5]; 2^f is a polynomial in f; the
// integer part goes straight into the exponent field.  n + K below -126 is clamped (the result is then a value below
// 2^-126 times a polynomial in a large |f|: nothing a sum of exponentials can see).  v must be finite.
constexpr float kExpMagic = 12582912.f;                  // 1.5 * 2^23: one unit in the last place is 1
constexpr float kExpMagicLow = kExpMagic - 126.f;
// Least-maximum-relative-error polynomials of 2^f on [-0.5, 0.5], scaled so that the mean relative error is zero.
// degree 2: |error| <= 1.8e-3 (row sums over thousands of keys: the errors average out), degree 4: <= 2.7e-6.
template <int DEG>
__device__ __forceinline__ uint64_t exp2_frac_poly(uint64_t f2) {
  if (DEG == 2) {
    const float c0 = 1.000384331f, c1 = 0.703401566f, c2 = 0.238411725f;
    return fma2(fma2(pack2(c2, c2), f2, pack2(c1, c1)), f2, pack2(c0, c0));
  } else if (DEG == 3) {
    const float c0 = 0.999922991f, c1 = 0.693257451f, c2 = 0.242609292f, c3 = 0.0551710390f;
    return fma2(fma2(fma2(pack2(c3, c3), f2, pack2(c2, c2)), f2, pack2(c1, c1)), f2, pack2(c0, c0));
  } else {
    const float c0 = 0.999999225f, c1 = 0.693121791f, c2 = 0.240247443f, c3 = 0.0559178069f, c4 = 0.00957006868f;
    return fma2(fma2(fma2(fma2(pack2(c4, c4), f2, pack2(c3, c3)), f2, pack2(c2, c2)), f2, pack2(c1, c1)), f2, pack2(c0, c0));
  }
}
// mk2 = (kExpMagic + K) twice.  Returns the pair 2^(v*c + K).
template <int DEG>
__device__ __forceinline__ uint64_t exp2_poly_pair(uint64_t v2, uint64_t c2, uint64_t mk2) {
  float t0, t1;
  unpack2(fma2(v2, c2, mk2), t0, t1);                    // magic + K + round(v*c)
  t0 = fmaxf(t0, kExpMagicLow);
  t1 = fmaxf(t1, kExpMagicLow);
  const uint64_t nr2 = sub2(mk2, pack2(t0, t1));         // -round(v*c)
  float p0, p1;
  unpack2(exp2_frac_poly<DEG>(fma2(v2, c2, nr2)), p0, p1);
  // (bits of t) << 23 = (n + K) << 23 modulo 2^32: added to the bits of p in [0.70, 1.42] it lowers the exponent by |n + K|
  p0 = __int_as_float(__float_as_int(p0) + (__float_as_int(t0) << 23));
  p1 = __int_as_float(__float_as_int(p1) + (__float_as_int(t1) << 23));
  return pack2(p0, p1);
}

__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// ---------------------------------------------------------------- host: tensor maps
// [tokens][heads][d] bf16 tensor with byte strides, viewed as (d, heads, tokens); box = 64 x 1 x rows.
inline bool make_tmap_rows(void* encode_fn, CUtensorMap* map, const void* base, uint64_t d, uint64_t heads,
                           uint64_t tokens, uint64_t head_stride_bytes, uint64_t token_stride_bytes, uint32_t box_rows) {
  if (encode_fn == nullptr || base == nullptr || tokens == 0 || heads == 0) return false;
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  const cuuint64_t dims[3] = {d, heads, tokens};
  const cuuint64_t strides[2] = {head_stride_bytes, token_stride_bytes};
  const cuuint32_t box[3] = {64, 1, box_rows};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult rc = reinterpret_cast<EncodeFn>(encode_fn)(
      map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
      CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS;
}

}  // namespace tc
}  // namespace mkv

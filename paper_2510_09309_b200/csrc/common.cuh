// Shared declarations of the MaskKV CUDA library (sm_100a): context, resolved problem shape,
// element loads.  Internal; the public surface is include/maskkv.h.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include "maskkv.h"

struct maskkv_ctx {
  int device;
  int sm_count;
  int smem_optin;          // max opt-in dynamic shared memory per block
  uint32_t* status_dev;    // 256-byte block; word 0 = status flags, word 1 = where a wait gave up
  void* encode_tiled;      // cuTensorMapEncodeTiled, resolved through the runtime
  unsigned long long launches;  // kernels launched through this context so far
  unsigned long long tc_launches;  // of those, kernels of the tcgen05 (tensor-core) paths
  int last_cuda_error;     // cudaError_t of the most recent failed runtime call (0 = none)
  uint32_t host_flags;     // status bits raised on the host (MASKKV_FLAG_FALLBACK); reported and cleared by maskkv_check_status
  unsigned force_simt;     // MASKKV_FORCE_SIMT, debugging: bit 0 = scoring sweep 1, bit 1 = scoring sweep 2, bit 2 = attention on the FP32 pipes
  int score_head_groups;   // MASKKV_SCORE_HEAD_GROUPS: scoring takes the KV heads in this many groups, both sweeps of a group back to
                           // back, so that sweep 2 finds the group's keys in L2 (1 = all heads at once)
  unsigned kernel_choice;  // MASKKV_KERNEL_CHOICE, debugging: bit 0 = projection on single CTAs instead of pairs, bit 1 / bit 2 / bit 3 = selection always on one CTA per segment with the keys in shared memory / always on clusters / always on one CTA per segment with the keys in registers, bit 5 / bit 6 = attention always / never with two units per CTA, bit 7 = selection always on the persistent kernel, bit 8 = that kernel on at most 3 CTAs
};

// The descriptor after validation, passed to kernels by value.
struct Shape {
  int dtype, H, Hkv, g, d, R;
  float scale;
  long long q_ts, q_hs, kv_ts, kv_hs;     // strides in elements
  const int32_t* prompt_cu;               // device
  const int32_t* live_cu;                 // device
  int sumN, sumM, maxN, maxM;
  int hk0, hkn;                           // KV heads [hk0, hk0 + hkn) a scoring launch covers (all of them unless the heads are taken in groups)
};

namespace mkv {

constexpr int kMaxAttrDevices = 64;   // per-device "attribute set" tables of the kernels that opt into large shared memory

// Programmatic dependent launch.  Every kernel of the layer path is launched with launch_overlapped(): its blocks may
// be scheduled while the previous kernel of the stream is still running, which hides the launch latency and the
// block's own set-up.  A kernel first lets its own successor go (pdl_launch_dependents), does whatever touches no
// global memory, then calls pdl_wait(), which returns once the previous kernel has completed and its writes are
// visible; every thread calls it before its first global access, so completion is transitive along the stream.
// Both are no-ops in a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// cluster_x > 1: thread-block clusters of that many CTAs along x (grid.x must be a multiple of it).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                             unsigned cluster_x, Args&&... args) {
  static const int serial = [] { const char* e = getenv("MASKKV_SERIAL_LAUNCH"); return e != nullptr && e[0] == '1'; }();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = serial ? 0 : 1;   // MASKKV_SERIAL_LAUNCH=1: ordinary stream order
  cfg.numAttrs = 1;
  if (cluster_x > 1) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  cfg.attrs = attr;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  return launch_overlapped_cluster(kernel, grid, block, smem, st, 1u, static_cast<Args&&>(args)...);
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Load `n` consecutive elements (n * sizeof(T) a multiple of 16, src 16-byte aligned) into floats.
template <int n>
__device__ __forceinline__ void load_row(const float* __restrict__ src, float* dst) {
#pragma unroll
  for (int c = 0; c < n; c += 4) {
    float4 v = *reinterpret_cast<const float4*>(src + c);
    dst[c] = v.x; dst[c + 1] = v.y; dst[c + 2] = v.z; dst[c + 3] = v.w;
  }
}
template <int n>
__device__ __forceinline__ void load_row(const __nv_bfloat16* __restrict__ src, float* dst) {
#pragma unroll
  for (int c = 0; c < n; c += 8) {
    uint4 v = *reinterpret_cast<const uint4*>(src + c);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      dst[c + 2 * t] = __uint_as_float(w[t] << 16);
      dst[c + 2 * t + 1] = __uint_as_float(w[t] & 0xffff0000u);
    }
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Request that owns row `row` of a cumulative array cu[0..R].
__device__ __forceinline__ int find_request(const int32_t* __restrict__ cu, int R, int row) {
  int lo = 0, hi = R;  // invariant: cu[lo] <= row < cu[hi]
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= row) lo = mid; else hi = mid;
  }
  return lo;
}

}  // namespace mkv

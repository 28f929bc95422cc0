// C ABI of the MaskKV library: argument validation, workspace carving and kernel launches.
// Every entry point validates first and launches nothing on failure (see include/maskkv.h).
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <nvtx3/nvToolsExt.h>

#include "attend_simt.cuh"
#include "attend_tc.h"
#include "budget.cuh"
#include "common.cuh"
#include "compact.cuh"
#include "importance.cuh"
#include "project_tc.h"
#include "refresh.cuh"
#include "score_simt.cuh"
#include "score_tc.h"
#include "select.cuh"
#include "selftest.h"

namespace {

struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() { if (switched) cudaSetDevice(prev); }
};

// A named range around every call that launches kernels: shows up in a profiler's timeline, costs a few nanoseconds
// when none is attached.
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int elem_size(int dtype) { return dtype == MASKKV_F32 ? 4 : 2; }

// Validates the descriptor and resolves defaults.  Returns MASKKV_OK or an error code.
int resolve(const maskkv_desc_t* d, Shape* sh) {
  if (d == nullptr) return MASKKV_E_INVALID;
  if (d->dtype != MASKKV_F32 && d->dtype != MASKKV_BF16) return MASKKV_E_UNSUPPORTED;
  if (d->head_dim != 64 && d->head_dim != 128) return MASKKV_E_UNSUPPORTED;
  if (d->n_q_heads <= 0 || d->n_kv_heads <= 0 || d->n_q_heads % d->n_kv_heads != 0) return MASKKV_E_INVALID;
  if (d->n_requests <= 0) return MASKKV_E_INVALID;
  if (d->prompt_cu == nullptr || d->live_cu == nullptr || d->prompt_cu_dev == nullptr || d->live_cu_dev == nullptr)
    return MASKKV_E_INVALID;
  if (d->prompt_cu[0] != 0 || d->live_cu[0] != 0) return MASKKV_E_INVALID;
  sh->dtype = d->dtype;
  sh->H = d->n_q_heads;
  sh->Hkv = d->n_kv_heads;
  sh->g = sh->H / sh->Hkv;
  sh->d = d->head_dim;
  sh->R = d->n_requests;
  sh->scale = d->softmax_scale > 0.f ? d->softmax_scale : (float)(1.0 / sqrt((double)d->head_dim));
  sh->maxN = sh->maxM = 0;
  for (int r = 0; r < sh->R; ++r) {
    const long long n = (long long)d->prompt_cu[r + 1] - d->prompt_cu[r];
    const long long m = (long long)d->live_cu[r + 1] - d->live_cu[r];
    if (n < 0 || m < 0) return MASKKV_E_INVALID;
    if (n > sh->maxN) sh->maxN = (int)n;
    if (m > sh->maxM) sh->maxM = (int)m;
  }
  sh->sumN = d->prompt_cu[sh->R];
  sh->sumM = d->live_cu[sh->R];
  sh->q_hs = d->q_head_stride > 0 ? d->q_head_stride : sh->d;
  sh->q_ts = d->q_token_stride > 0 ? d->q_token_stride : (long long)sh->H * sh->q_hs;
  sh->kv_hs = d->kv_head_stride > 0 ? d->kv_head_stride : sh->d;
  sh->kv_ts = d->kv_token_stride > 0 ? d->kv_token_stride : (long long)sh->Hkv * sh->kv_hs;
  const long long es = elem_size(sh->dtype);
  if ((sh->q_hs * es) % 16 || (sh->q_ts * es) % 16 || (sh->kv_hs * es) % 16 || (sh->kv_ts * es) % 16) return MASKKV_E_ALIGN;
  if (sh->q_hs < sh->d || sh->kv_hs < sh->d) return MASKKV_E_INVALID;
  if ((reinterpret_cast<uintptr_t>(d->prompt_cu_dev) & 3u) || (reinterpret_cast<uintptr_t>(d->live_cu_dev) & 3u)) return MASKKV_E_ALIGN;
  sh->prompt_cu = d->prompt_cu_dev;
  sh->live_cu = d->live_cu_dev;
  sh->hk0 = 0;
  sh->hkn = sh->Hkv;
  return MASKKV_OK;
}

struct ScoreWorkspace {
  size_t lse_off, part_off, mass_off, cnt_off, col_off, total;
  int C, Tmax;
};

// KV heads per scoring launch: all of them, or Hkv / groups when the context takes the heads in groups (only the plain
// case - one query head per KV head, at most 256 voters per request - is ever grouped).
int score_heads_per_launch(const maskkv_ctx* ctx, const Shape& sh) {
  if (ctx == nullptr || ctx->score_head_groups <= 1 || mkv::tc::score_tc_split_blocks(sh) || !mkv::tc::score_tc_supported(ctx, sh) ||
      (ctx->force_simt & 3u))
    return sh.Hkv;
  const int groups = ctx->score_head_groups < sh.Hkv ? ctx->score_head_groups : sh.Hkv;
  return (sh.Hkv + groups - 1) / groups;
}

ScoreWorkspace score_workspace(const maskkv_ctx* ctx, const Shape& sh) {
  ScoreWorkspace w;
  const long long keys = (long long)sh.maxN + sh.maxM;
  w.C = (int)((keys + mkv::kStatsChunk - 1) / mkv::kStatsChunk);
  if (ctx != nullptr) {
    Shape per_launch = sh;
    per_launch.hkn = score_heads_per_launch(ctx, sh);
    if (w.C < mkv::tc::score_tc_max_chunks(ctx, per_launch)) w.C = mkv::tc::score_tc_max_chunks(ctx, per_launch);
  }
  if (w.C < 1) w.C = 1;
  w.Tmax = mkv::tc::score_tc_max_tiles(sh);               // >= ceil(keys / 128), the FP32-pipe kernel's tiling
  if (w.Tmax < 1) w.Tmax = 1;
  size_t off = 0;
  w.lse_off = off;  off = align_up(off + sizeof(float) * (size_t)sh.H * sh.sumM, 256);
  w.part_off = off; off = align_up(off + sizeof(float2) * (size_t)sh.H * sh.sumM * w.C, 256);
  w.mass_off = off; off = align_up(off + sizeof(float2) * (size_t)sh.R * sh.Hkv * w.Tmax * 8, 256);
  w.cnt_off = off;  off = align_up(off + sizeof(uint32_t) * (size_t)sh.R * sh.Hkv, 256);
  w.col_off = off;  off = align_up(off + mkv::tc::score_tc_colpart_bytes(sh), 256);   // per-block column sums (grouped heads)
  w.total = off;
  return w;
}

// Adds `n` launches to the context's counter and maps the runtime's launch status to a return code.
inline int launch_status(maskkv_ctx* ctx, int n) {
  ctx->launches += (unsigned long long)n;
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) ctx->last_cuda_error = (int)e;
  return e == cudaSuccess ? MASKKV_OK : MASKKV_E_CUDA;
}

// Scoring = sweep 1 (row statistics) + merge + sweep 2 (column sums) + mass reduction.  bf16 problems run the two
// sweeps on the tensor cores; fp32 problems (and anything the tensor-core path cannot take) on the FP32 pipes.
template <typename T, int D>
int launch_score(maskkv_ctx* ctx, const Shape& sh, const maskkv_desc_t* desc, const ScoreWorkspace& w, bool any_without_voters,
                 const void* q, const void* kp, const void* km, const float* rw, float* scores, float* scores_live, float* mass_p,
                 float* mass_m, unsigned char* ws, cudaStream_t st) {
  float* lse = reinterpret_cast<float*>(ws + w.lse_off);
  float2* part = reinterpret_cast<float2*>(ws + w.part_off);
  float2* mass_part = reinterpret_cast<float2*>(ws + w.mass_off);
  uint32_t* seg_cnt = reinterpret_cast<uint32_t*>(ws + w.cnt_off);
  const int S = sh.R * sh.Hkv;
  const bool tc_ok = mkv::tc::score_tc_supported(ctx, sh);
  const bool want_tc2 = tc_ok && !(ctx->force_simt & 2u);
  int n = 0;
  const int per_launch = score_heads_per_launch(ctx, sh);
  if (per_launch < sh.Hkv && sh.sumM > 0) {
    // The KV heads in groups, both sweeps of a group back to back: the group's keys (per_launch x N x 2d bytes) are
    // still in L2 when sweep 2 asks for them, so the key tensor crosses the memory bus once instead of twice.
    for (int hk0 = 0; hk0 < sh.Hkv; hk0 += per_launch) {
      Shape g = sh;
      g.hk0 = hk0;
      g.hkn = sh.Hkv - hk0 < per_launch ? sh.Hkv - hk0 : per_launch;
      int launched = 0;
      if (mkv::tc::launch_score_stats_tc(ctx, g, desc->prompt_cu, desc->live_cu, q, kp, km, part, w.C, seg_cnt, st) != 0) {
        launch_status(ctx, n);
        return MASKKV_E_CUDA;
      }
      ++n; ++ctx->tc_launches;
      if (mkv::tc::launch_score_colsum_tc(ctx, g, desc->prompt_cu, desc->live_cu, q, kp, km, lse, part, w.C, rw, scores,
                                          reinterpret_cast<float*>(ws + w.col_off), mass_part, w.Tmax, seg_cnt, mass_p, mass_m, scores_live,
                                          any_without_voters, st, &launched) != 0) {
        launch_status(ctx, n + launched);
        return MASKKV_E_CUDA;
      }
      n += launched; ++ctx->tc_launches;
    }
    return launch_status(ctx, n);
  }
  bool tc1 = false;                                          // sweep 1 ran on the tensor cores: `part` has its layout
  if (sh.sumM > 0) {
    if (tc_ok && !(ctx->force_simt & 1u))
      tc1 = mkv::tc::launch_score_stats_tc(ctx, sh, desc->prompt_cu, desc->live_cu, q, kp, km, part, w.C, seg_cnt, st) == 0;
    if (tc1) { ++ctx->tc_launches; ++n; }
    else if (tc_ok && !(ctx->force_simt & 1u)) ctx->host_flags |= MASKKV_FLAG_FALLBACK;   // nobody asked for the FP32 pipes
    if (!tc1) {
      const int q_tiles = (sh.maxM + mkv::kSimtThreads - 1) / mkv::kSimtThreads;
      dim3 g1((unsigned)((sh.maxN + sh.maxM + mkv::kStatsChunk - 1) / mkv::kStatsChunk), sh.H, sh.R * q_tiles);
      mkv::score_stats_simt<T, D><<<g1, mkv::kSimtThreads, 0, st>>>(sh, (const T*)q, (const T*)kp, (const T*)km, part, w.C);
      const long long rows = (long long)sh.H * sh.sumM;
      mkv::score_merge_stats<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(sh, part, w.C, lse);
      n += 2;
      if (want_tc2 && cudaMemsetAsync(seg_cnt, 0, sizeof(uint32_t) * (size_t)S, st) != cudaSuccess) return launch_status(ctx, n);
    }
  }
  bool tc2 = false;
  if (want_tc2) {
    // after a tensor-core sweep 1 the kernel merges the partials itself; otherwise it reads lse
    int launched = 0;
    float* colpart = reinterpret_cast<float*>(ws + w.col_off);
    tc2 = mkv::tc::launch_score_colsum_tc(ctx, sh, desc->prompt_cu, desc->live_cu, q, kp, km, lse, tc1 ? part : nullptr, w.C, rw,
                                          scores, colpart, mass_part, w.Tmax, seg_cnt, mass_p, mass_m, scores_live, any_without_voters, st,
                                          &launched) == 0;
    if (!tc2) { ctx->host_flags |= MASKKV_FLAG_FALLBACK; n += launched; }
    if (tc2) {
      ++ctx->tc_launches;
      n += launched;
      if (mkv::tc::score_tc_split_blocks(sh)) {              // the masses of the per-block path are summed here
        mkv::score_mass_reduce<<<(S + 3) / 4, 128, 0, st>>>(sh, mass_part, w.Tmax, mass_p, mass_m);
        ++n;
      }
    }
  }
  if (!tc2) {
    if (tc1) { mkv::tc::launch_score_merge_tc(ctx, sh, desc->prompt_cu, desc->live_cu, part, w.C, lse, st); ++n; }
    dim3 g2(w.Tmax, sh.Hkv, sh.R);
    mkv::score_colsum_simt<T, D><<<g2, mkv::kSimtThreads, 0, st>>>(sh, (const T*)q, (const T*)kp, (const T*)km, lse, rw,
                                                                    scores, scores_live, mass_part, w.Tmax);
    mkv::score_mass_reduce<<<(S + 3) / 4, 128, 0, st>>>(sh, mass_part, w.Tmax, mass_p, mass_m);
    n += 2;
  }
  return launch_status(ctx, n);
}

template <typename T, int D>
int launch_attend_simt(maskkv_ctx* ctx, const Shape& sh, const void* q, const int32_t* q_cu, int sum_q, int max_q, const void* kl,
                       const void* vl, const void* kc, const void* vc, const int32_t* offsets, long long capacity, void* out, float* lse,
                       cudaStream_t st) {
  if (max_q == 0) return MASKKV_OK;
  dim3 grid((max_q + mkv::kAttendWarps - 1) / mkv::kAttendWarps, sh.H, sh.R);
  mkv::attend_simt<T, D><<<grid, mkv::kAttendWarps * 32, 0, st>>>(sh, (const T*)q, (const T*)kl, (const T*)vl, (const T*)kc,
                                                                   (const T*)vc, offsets, q_cu, sum_q, capacity, (T*)out, lse,
                                                                   ctx->status_dev);
  return launch_status(ctx, 1);
}

// ---- scratch for maskkv_score_noalloc -------------------------------------------------------------------
// Lives in the library image: every GPU that loads the library holds these bytes until the process exits.
constexpr size_t kStaticScratchBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static void* g_static_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of g_static_scratch on `device`.  In host code the array's name is only a handle for the
// runtime, never an address a kernel may use, so it is resolved once per device (with that device current).
int static_scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return MASKKV_E_UNSUPPORTED;
  if (g_static_scratch_ptr[device] == nullptr) {
    DeviceGuard guard(device);
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return MASKKV_E_CUDA;
    }
    g_static_scratch_ptr[device] = p;
  }
  *out = g_static_scratch_ptr[device];
  return MASKKV_OK;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

const char* maskkv_status_string(int code) {
  switch (code) {
    case MASKKV_OK: return "ok";
    case MASKKV_E_INVALID: return "invalid argument";
    case MASKKV_E_UNSUPPORTED: return "unsupported dtype, head_dim or device";
    case MASKKV_E_ALIGN: return "pointer or stride not 16-byte aligned";
    case MASKKV_E_WORKSPACE: return "workspace missing or too small";
    case MASKKV_E_CAPACITY: return "capacity too small";
    case MASKKV_E_CUDA: return "CUDA call failed";
    case MASKKV_E_TIMEOUT: return "a bounded device wait expired";
    default: return "unknown status";
  }
}

int maskkv_create(maskkv_ctx** out, int device) {
  if (out == nullptr) return MASKKV_E_INVALID;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return MASKKV_E_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return MASKKV_E_CUDA;
  if (prop.major != 10) return MASKKV_E_UNSUPPORTED;
  DeviceGuard guard(device);
  maskkv_ctx* ctx = static_cast<maskkv_ctx*>(calloc(1, sizeof(maskkv_ctx)));
  if (ctx == nullptr) return MASKKV_E_INVALID;
  ctx->device = device;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->smem_optin = (int)prop.sharedMemPerBlockOptin;
  if (cudaMalloc(&ctx->status_dev, 256) != cudaSuccess || cudaMemset(ctx->status_dev, 0, 256) != cudaSuccess) {
    free(ctx);
    return MASKKV_E_CUDA;
  }
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ctx->encode_tiled, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    ctx->encode_tiled = nullptr;
  if (const char* e = getenv("MASKKV_FORCE_SIMT")) ctx->force_simt = (unsigned)strtoul(e, nullptr, 0);
  if (const char* e = getenv("MASKKV_KERNEL_CHOICE")) ctx->kernel_choice = (unsigned)strtoul(e, nullptr, 0);
  ctx->score_head_groups = 1;
  if (const char* e = getenv("MASKKV_SCORE_HEAD_GROUPS")) ctx->score_head_groups = (int)strtol(e, nullptr, 0);
  cudaFuncSetAttribute(mkv::select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->smem_optin - mkv::kSelectStaticSmem);
  cudaFuncSetAttribute(mkv::select_kernel_cta, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->smem_optin - mkv::kSelectStaticSmem);
  cudaFuncSetAttribute(mkv::select_kernel_stream, cudaFuncAttributeMaxDynamicSharedMemorySize, mkv::kSelectStreamSmem);
  cudaFuncSetAttribute(mkv::budget_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
  cudaFuncSetAttribute(mkv::select_kernel_reg<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, mkv::kSelectCandCap * 4);
  cudaFuncSetAttribute(mkv::select_kernel_reg<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, mkv::kSelectCandCap * 4);
  if (cudaGetLastError() != cudaSuccess) { cudaFree(ctx->status_dev); free(ctx); return MASKKV_E_CUDA; }
  *out = ctx;
  return MASKKV_OK;
}

int maskkv_destroy(maskkv_ctx* ctx) {
  if (ctx == nullptr) return MASKKV_E_INVALID;
  DeviceGuard guard(ctx->device);
  cudaFree(ctx->status_dev);
  free(ctx);
  return MASKKV_OK;
}

int maskkv_check_status(maskkv_ctx* ctx, void* stream, uint32_t* flags_out) {
  if (ctx == nullptr) return MASKKV_E_INVALID;
  DeviceGuard guard(ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t flags = 0;
  if (cudaMemcpyAsync(&flags, ctx->status_dev, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MASKKV_E_CUDA;
  if (cudaMemsetAsync(ctx->status_dev, 0, 8, st) != cudaSuccess) return MASKKV_E_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MASKKV_E_CUDA;
  flags |= ctx->host_flags;
  ctx->host_flags = 0;
  if (flags_out) *flags_out = flags;
  return (flags & MASKKV_FLAG_TIMEOUT) ? MASKKV_E_TIMEOUT : MASKKV_OK;
}

int maskkv_selftest_wait_expiry(maskkv_ctx* ctx, void* stream) {
  if (ctx == nullptr) return MASKKV_E_INVALID;
  DeviceGuard guard(ctx->device);
  mkv::tc::launch_wait_expiry_selftest(ctx, static_cast<cudaStream_t>(stream));
  return launch_status(ctx, 1);
}

int maskkv_selftest_exp_rate(maskkv_ctx* ctx, int iters, float* scratch_dev, int64_t* n_exp_out, void* stream) {
  if (ctx == nullptr || scratch_dev == nullptr || n_exp_out == nullptr || iters <= 0 || iters > (1 << 20)) return MASKKV_E_INVALID;
  DeviceGuard guard(ctx->device);
  *n_exp_out = mkv::tc::launch_ex2_rate_selftest(ctx, scratch_dev, iters, static_cast<cudaStream_t>(stream));
  return launch_status(ctx, 1);
}

uint64_t maskkv_launch_count(const maskkv_ctx* ctx) { return ctx ? ctx->launches : 0; }
const char* maskkv_last_cuda_error(const maskkv_ctx* ctx) {
  return ctx && ctx->last_cuda_error ? cudaGetErrorString((cudaError_t)ctx->last_cuda_error) : "";
}
uint64_t maskkv_tensor_core_launch_count(const maskkv_ctx* ctx) { return ctx ? ctx->tc_launches : 0; }

size_t maskkv_workspace_bytes(const maskkv_ctx* ctx, const maskkv_desc_t* desc) {
  (void)ctx;
  Shape sh;
  if (resolve(desc, &sh) != MASKKV_OK) return 0;
  return score_workspace(ctx, sh).total;
}

int maskkv_layer_budgets(int64_t k_p, double beta, int32_t n_layers, const double* importance_host,
                         const uint8_t* is_boundary_host, int32_t* k_l_out_host) {
  if (n_layers <= 0 || importance_host == nullptr || k_l_out_host == nullptr || k_p < 0) return MASKKV_E_INVALID;
  if (!(beta >= 0.0 && beta <= 1.0)) return MASKKV_E_INVALID;
  // volatile keeps every intermediate a rounded double (no contraction, no extended precision)
  volatile double base_real = beta * (double)k_p;
  base_real = base_real / (double)n_layers;
  const long long k_base = (long long)floor(base_real + 1e-6);                  // Eq. 9
  const long long k_imp = k_p - (long long)n_layers * k_base;                   // Eq. 10
  volatile double i_b = 0.0, i_m = 0.0;
  int n_b = 0;
  for (int l = 0; l < n_layers; ++l) {
    const bool bnd = is_boundary_host ? is_boundary_host[l] != 0 : (l == 0 || l == n_layers - 1);
    if (bnd) { i_b = i_b + importance_host[l]; ++n_b; } else { i_m = i_m + importance_host[l]; }
  }
  const int n_m = n_layers - n_b;
  volatile double denom = i_b + i_m;
  volatile double group_b = 0.0;
  if (denom > 0.0) { group_b = (double)k_imp * i_b; group_b = group_b / denom; } // Eq. 11
  volatile double group_m = (double)k_imp - group_b;                            // Eq. 12
  for (int l = 0; l < n_layers; ++l) {                                          // Eq. 13
    const bool bnd = is_boundary_host ? is_boundary_host[l] != 0 : (l == 0 || l == n_layers - 1);
    volatile double share = bnd ? group_b / (double)(n_b > 0 ? n_b : 1) : group_m / (double)(n_m > 0 ? n_m : 1);
    k_l_out_host[l] = (int32_t)(k_base + (long long)floor(share + 1e-6));
  }
  return MASKKV_OK;
}

size_t maskkv_layer_importance_workspace_bytes(const maskkv_ctx* ctx) {
  return ctx ? sizeof(double) * (size_t)ctx->sm_count * mkv::kImpBlocksPerSm : 0;
}

int maskkv_layer_importance(maskkv_ctx* ctx, int32_t dtype, const void* h_in_dev, const void* h_out_dev, int64_t n_tokens,
                            int32_t hidden, int64_t in_row_stride, int64_t out_row_stride, float* importance_out_dev,
                            void* workspace_dev, size_t workspace_bytes, void* stream) {
  TraceRange trace("maskkv_layer_importance");
  if (ctx == nullptr || importance_out_dev == nullptr || n_tokens < 0 || hidden <= 0) return MASKKV_E_INVALID;
  if (dtype != MASKKV_F32 && dtype != MASKKV_BF16) return MASKKV_E_UNSUPPORTED;
  if (n_tokens > 0 && (h_in_dev == nullptr || h_out_dev == nullptr)) return MASKKV_E_INVALID;
  const int es = elem_size(dtype);
  if (in_row_stride <= 0) in_row_stride = hidden;
  if (out_row_stride <= 0) out_row_stride = hidden;
  if (in_row_stride < hidden || out_row_stride < hidden) return MASKKV_E_INVALID;
  if (((long long)hidden * es) % 16 || (in_row_stride * es) % 16 || (out_row_stride * es) % 16 || !aligned16(h_in_dev) ||
      !aligned16(h_out_dev) || (reinterpret_cast<uintptr_t>(workspace_dev) & 7u))
    return MASKKV_E_ALIGN;
  if (workspace_dev == nullptr || workspace_bytes < maskkv_layer_importance_workspace_bytes(ctx)) return MASKKV_E_WORKSPACE;
  DeviceGuard guard(ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int rows_per_block = mkv::kImpThreads / 32;
  long long blocks = (n_tokens + rows_per_block - 1) / rows_per_block;
  const long long max_blocks = (long long)ctx->sm_count * mkv::kImpBlocksPerSm;
  if (blocks > max_blocks) blocks = max_blocks;
  if (blocks < 1) blocks = 1;
  double* partial = static_cast<double*>(workspace_dev);
  if (dtype == MASKKV_F32)
    mkv::importance_partial_kernel<float><<<(unsigned)blocks, mkv::kImpThreads, 0, st>>>(
        static_cast<const float*>(h_in_dev), static_cast<const float*>(h_out_dev), n_tokens, hidden, in_row_stride, out_row_stride, partial);
  else
    mkv::importance_partial_kernel<__nv_bfloat16><<<(unsigned)blocks, mkv::kImpThreads, 0, st>>>(
        static_cast<const __nv_bfloat16*>(h_in_dev), static_cast<const __nv_bfloat16*>(h_out_dev), n_tokens, hidden, in_row_stride,
        out_row_stride, partial);
  mkv::importance_final_kernel<<<1, mkv::kImpThreads, 0, st>>>(partial, (int)blocks, n_tokens, importance_out_dev);
  return launch_status(ctx, 2);
}

int maskkv_refresh_set(maskkv_ctx* ctx, int32_t dtype, const void* v_cur_dev, const void* v_prev_dev, int64_t n_tokens,
                       int32_t width, int64_t cur_row_stride, int64_t prev_row_stride, float delta, int32_t refresh_all,
                       float* cos_out_dev, int32_t* idx_out_dev, int32_t* count_out_dev, void* stream) {
  TraceRange trace("maskkv_refresh_set");
  if (ctx == nullptr || idx_out_dev == nullptr || count_out_dev == nullptr) return MASKKV_E_INVALID;
  if (dtype != MASKKV_F32 && dtype != MASKKV_BF16) return MASKKV_E_UNSUPPORTED;
  if (n_tokens < 0 || n_tokens > 0x7fffffffLL || width <= 0 || !(delta == delta)) return MASKKV_E_INVALID;
  const int es = elem_size(dtype);
  if (cur_row_stride == 0) cur_row_stride = width;
  if (prev_row_stride == 0) prev_row_stride = width;
  if (cur_row_stride < width || prev_row_stride < width) return MASKKV_E_INVALID;
  const bool reads = !refresh_all || cos_out_dev != nullptr;
  if (reads && n_tokens > 0) {
    if (v_cur_dev == nullptr || v_prev_dev == nullptr) return MASKKV_E_INVALID;
    if (((long long)width * es) % 16 != 0 || (cur_row_stride * es) % 16 != 0 || (prev_row_stride * es) % 16 != 0 ||
        !aligned16(v_cur_dev) || !aligned16(v_prev_dev))
      return MASKKV_E_ALIGN;
  }
  DeviceGuard guard(ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int n = 0;
  if (n_tokens > 0) {
    const int rows_per_block = mkv::kRefreshThreads / 32;
    long long blocks = (n_tokens + rows_per_block - 1) / rows_per_block;
    const long long max_blocks = (long long)ctx->sm_count * 8;
    if (blocks > max_blocks) blocks = max_blocks;
    if (dtype == MASKKV_F32)
      mkv::refresh_flag_kernel<float><<<(unsigned)blocks, mkv::kRefreshThreads, 0, st>>>(
          static_cast<const float*>(v_cur_dev), static_cast<const float*>(v_prev_dev), n_tokens, width, cur_row_stride,
          prev_row_stride, delta, refresh_all ? 1 : 0, cos_out_dev, idx_out_dev);
    else
      mkv::refresh_flag_kernel<__nv_bfloat16><<<(unsigned)blocks, mkv::kRefreshThreads, 0, st>>>(
          static_cast<const __nv_bfloat16*>(v_cur_dev), static_cast<const __nv_bfloat16*>(v_prev_dev), n_tokens, width,
          cur_row_stride, prev_row_stride, delta, refresh_all ? 1 : 0, cos_out_dev, idx_out_dev);
    ++n;
  }
  mkv::launch_overlapped(mkv::refresh_compact_kernel, dim3(1), dim3(mkv::kRefreshScanThreads), 0, st, (long long)n_tokens, idx_out_dev,
                         count_out_dev);
  return launch_status(ctx, n + 1);
}

size_t maskkv_mask_project_workspace_bytes(int64_t n_mask, int32_t width) {
  return n_mask > 0 && width > 0 ? align_up((size_t)n_mask * (size_t)width * 2, 256) : 0;
}

int maskkv_mask_project(maskkv_ctx* ctx, int32_t dtype, const void* hidden_dev, int64_t n_tokens, int32_t width,
                        int64_t hidden_row_stride, const int32_t* positions_dev, int32_t n_mask, const void* w_vocab_dev,
                        int32_t vocab, int64_t w_row_stride, int32_t out_dtype, void* logits_out_dev, int64_t out_row_stride,
                        void* workspace_dev, size_t workspace_bytes, void* stream) {
  TraceRange trace("maskkv_mask_project");
  if (ctx == nullptr || n_mask < 0 || n_tokens < 0 || width <= 0 || vocab <= 0) return MASKKV_E_INVALID;
  if (dtype != MASKKV_BF16 || (out_dtype != MASKKV_F32 && out_dtype != MASKKV_BF16)) return MASKKV_E_UNSUPPORTED;
  if (!mkv::tc::project_tc_supported(ctx)) return MASKKV_E_UNSUPPORTED;
  if (n_mask == 0) return MASKKV_OK;
  if (hidden_dev == nullptr || w_vocab_dev == nullptr || logits_out_dev == nullptr) return MASKKV_E_INVALID;
  if (positions_dev == nullptr && n_mask > n_tokens) return MASKKV_E_INVALID;
  if (hidden_row_stride == 0) hidden_row_stride = width;
  if (w_row_stride == 0) w_row_stride = width;
  if (out_row_stride == 0) out_row_stride = vocab;
  if (hidden_row_stride < width || w_row_stride < width || out_row_stride < vocab) return MASKKV_E_INVALID;
  const int out_vec = out_dtype == MASKKV_F32 ? 4 : 8;
  if (width % 8 || hidden_row_stride % 8 || w_row_stride % 8 || out_row_stride % out_vec || !aligned16(hidden_dev) ||
      !aligned16(w_vocab_dev) || !aligned16(logits_out_dev) || (reinterpret_cast<uintptr_t>(positions_dev) & 3u))
    return MASKKV_E_ALIGN;
  if (positions_dev != nullptr) {
    if (workspace_dev == nullptr || workspace_bytes < maskkv_mask_project_workspace_bytes(n_mask, width)) return MASKKV_E_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) return MASKKV_E_ALIGN;
  }
  DeviceGuard guard(ctx->device);
  int n = 0;
  if (mkv::tc::launch_project_tc(ctx, hidden_dev, n_tokens, width, hidden_row_stride, positions_dev, n_mask, w_vocab_dev, vocab,
                                 w_row_stride, logits_out_dev, out_row_stride, out_dtype == MASKKV_BF16 ? 1 : 0, workspace_dev,
                                 static_cast<cudaStream_t>(stream), &n) != 0) {
    ctx->launches += (unsigned long long)n;
    ctx->last_cuda_error = (int)cudaGetLastError();
    return MASKKV_E_CUDA;
  }
  return launch_status(ctx, n);
}

int maskkv_score(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* q_mask_dev, const void* k_prompt_dev,
                 const void* k_mask_dev, const float* row_weights_dev, float* scores_dev, float* mass_p_dev,
                 float* mass_m_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
  return maskkv_score_all_keys(ctx, desc, q_mask_dev, k_prompt_dev, k_mask_dev, row_weights_dev, scores_dev, nullptr, mass_p_dev,
                               mass_m_dev, workspace_dev, workspace_bytes, stream);
}

int maskkv_score_all_keys(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* q_mask_dev, const void* k_prompt_dev,
                          const void* k_mask_dev, const float* row_weights_dev, float* scores_dev, float* scores_live_dev,
                          float* mass_p_dev, float* mass_m_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
  TraceRange trace("maskkv_score_all_keys");
  if (ctx == nullptr) return MASKKV_E_INVALID;
  Shape sh;
  int rc = resolve(desc, &sh);
  if (rc != MASKKV_OK) return rc;
  if ((scores_dev == nullptr && sh.sumN > 0) || mass_p_dev == nullptr || mass_m_dev == nullptr) return MASKKV_E_INVALID;
  if (reinterpret_cast<uintptr_t>(scores_live_dev) & 3u) return MASKKV_E_ALIGN;
  if ((sh.sumM > 0 && (q_mask_dev == nullptr || k_mask_dev == nullptr)) || (sh.sumN > 0 && k_prompt_dev == nullptr))
    return MASKKV_E_INVALID;
  if (!aligned16(q_mask_dev) || !aligned16(k_prompt_dev) || !aligned16(k_mask_dev) || !aligned16(scores_dev) ||
      !aligned16(workspace_dev))
    return MASKKV_E_ALIGN;
  const ScoreWorkspace w = score_workspace(ctx, sh);
  if (workspace_dev == nullptr || workspace_bytes < w.total) return MASKKV_E_WORKSPACE;
  DeviceGuard guard(ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace_dev);
  bool any_without_voters = false;
  for (int r = 0; r < sh.R; ++r) any_without_voters |= desc->live_cu[r + 1] == desc->live_cu[r];
#define MKV_SCORE(T, D) launch_score<T, D>(ctx, sh, desc, w, any_without_voters, q_mask_dev, k_prompt_dev, k_mask_dev, row_weights_dev, scores_dev, \
                                                scores_live_dev, mass_p_dev, mass_m_dev, ws, st)
  if (sh.dtype == MASKKV_F32) return sh.d == 64 ? MKV_SCORE(float, 64) : MKV_SCORE(float, 128);
  return sh.d == 64 ? MKV_SCORE(__nv_bfloat16, 64) : MKV_SCORE(__nv_bfloat16, 128);
#undef MKV_SCORE
}

int maskkv_score_noalloc(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* q_mask_dev, const void* k_prompt_dev,
                         const void* k_mask_dev, const float* row_weights_dev, float* scores_dev, float* mass_p_dev,
                         float* mass_m_dev, void* stream) {
  if (ctx == nullptr) return MASKKV_E_INVALID;
  Shape sh;
  int rc = resolve(desc, &sh);
  if (rc != MASKKV_OK) return rc;
  const size_t need = maskkv_workspace_bytes(ctx, desc);
  if (need > kStaticScratchBytes) return MASKKV_E_WORKSPACE;   // problem too large for the built-in scratch
  void* scratch = nullptr;
  rc = static_scratch_address(ctx->device, &scratch);
  if (rc != MASKKV_OK) return rc;
  // Every scratch word the scoring kernels read is written earlier in the same call, so nothing has to be cleared.
  return maskkv_score(ctx, desc, q_mask_dev, k_prompt_dev, k_mask_dev, row_weights_dev, scores_dev, mass_p_dev, mass_m_dev,
                      scratch, kStaticScratchBytes, stream);
}

size_t maskkv_score_noalloc_max_bytes(void) { return kStaticScratchBytes; }

int maskkv_budget(maskkv_ctx* ctx, const maskkv_desc_t* desc, int32_t k_l, const int32_t* k_l_per_request_dev,
                  double alpha, const float* mass_p_dev, const float* mass_m_dev, int64_t capacity,
                  int32_t* budgets_dev, int32_t* offsets_dev, void* stream) {
  TraceRange trace("maskkv_budget");
  if (ctx == nullptr) return MASKKV_E_INVALID;
  Shape sh;
  int rc = resolve(desc, &sh);
  if (rc != MASKKV_OK) return rc;
  if (mass_p_dev == nullptr || mass_m_dev == nullptr || budgets_dev == nullptr || offsets_dev == nullptr) return MASKKV_E_INVALID;
  if (k_l < 0 || capacity < 0 || capacity > 0x7fffffffLL || !(alpha >= 0.0 && alpha <= 1.0)) return MASKKV_E_INVALID;
  const int S = sh.R * sh.Hkv;
  if (S > mkv::kBudgetMaxSegments) return MASKKV_E_UNSUPPORTED;
  DeviceGuard guard(ctx->device);
  const size_t smem = sizeof(double) * (S + sh.R) + sizeof(int) * S;
  mkv::launch_overlapped(mkv::budget_kernel, dim3(1), dim3(mkv::kBudgetThreads), smem, static_cast<cudaStream_t>(stream),
                         sh, k_l, k_l_per_request_dev, alpha, 1.0 - alpha, mass_p_dev, mass_m_dev, (long long)capacity, budgets_dev,
                         offsets_dev, ctx->status_dev);
  return launch_status(ctx, 1);
}

int maskkv_select(maskkv_ctx* ctx, const maskkv_desc_t* desc, const float* scores_dev, const int32_t* budgets_dev,
                  const int32_t* offsets_dev, int32_t* kept_idx_dev, void* workspace_dev, size_t workspace_bytes,
                  void* stream) {
  TraceRange trace("maskkv_select");
  (void)workspace_dev; (void)workspace_bytes;
  if (ctx == nullptr) return MASKKV_E_INVALID;
  Shape sh;
  int rc = resolve(desc, &sh);
  if (rc != MASKKV_OK) return rc;
  if (scores_dev == nullptr || budgets_dev == nullptr || offsets_dev == nullptr || kept_idx_dev == nullptr) return MASKKV_E_INVALID;
  if (!aligned16(scores_dev) || !aligned16(kept_idx_dev) || (reinterpret_cast<uintptr_t>(budgets_dev) & 3u) ||
      (reinterpret_cast<uintptr_t>(offsets_dev) & 3u))
    return MASKKV_E_ALIGN;
  DeviceGuard guard(ctx->device);
  const int cta_cache = (ctx->smem_optin - mkv::kSelectStaticSmem) / 4 - mkv::kSelectCtaCand;
  const int sel_force = (ctx->kernel_choice & 2u) ? 2 : (ctx->kernel_choice & 4u) ? 1 : (ctx->kernel_choice & 8u) ? 3 : 0;   // debugging: pin the kernel
  // more segments than one wave of clusters (two CTAs per SM): one CTA per segment gets through faster - with the keys in
  // registers up to 32768 scores per segment, staged in shared memory beyond that
  const bool batch = (long long)sh.R * sh.Hkv * mkv::kSelectCluster > 2LL * ctx->sm_count;
  // more segments than SMs: persistent CTAs, the next segment's scores copied to shared memory under the current one's work
  const bool stream_forced = (ctx->kernel_choice & 128u) != 0;
  if (sh.maxN <= mkv::kSelectBlockKeys && ((sel_force == 0 && sh.R * sh.Hkv > ctx->sm_count) || stream_forced)) {
    int grid = sh.R * sh.Hkv < ctx->sm_count ? sh.R * sh.Hkv : ctx->sm_count;
    if ((ctx->kernel_choice & 256u) && grid > 3) grid = 3;                     // debugging: several segments per CTA on small cases
    mkv::launch_overlapped(mkv::select_kernel_stream, dim3(grid), dim3(mkv::kSelectBlockThreads), mkv::kSelectStreamSmem,
                           static_cast<cudaStream_t>(stream), sh, scores_dev, budgets_dev, offsets_dev, kept_idx_dev, ctx->status_dev);
    return launch_status(ctx, 1);
  }
  // up to 32768 scores per segment: one CTA per segment with the keys in registers, also for one layer's few segments
  // (measured per layer, 32 segments of 32768 / 4096 scores: 10.2 / 8.1 us against 12.3 / 9.6 us on clusters)
  if (sh.maxN <= mkv::kSelectBlockKeys && (sel_force == 0 || sel_force == 3)) {
    mkv::launch_overlapped(mkv::select_kernel_block, dim3(sh.R * sh.Hkv), dim3(mkv::kSelectBlockThreads), 0,
                           static_cast<cudaStream_t>(stream), sh, scores_dev, budgets_dev, offsets_dev, kept_idx_dev, ctx->status_dev);
    return launch_status(ctx, 1);
  }
  if (sh.maxN <= cta_cache && ((batch && sel_force == 0) || sel_force == 2 || sh.maxN > mkv::kSelectRegKeys)) {
    const int n_cache = (sh.maxN + 3) & ~3;
    mkv::launch_overlapped(mkv::select_kernel_cta, dim3(sh.R * sh.Hkv), dim3(mkv::kSelectThreads),
                           (size_t)(n_cache + mkv::kSelectCtaCand) * 4, static_cast<cudaStream_t>(stream), sh, scores_dev, budgets_dev,
                           offsets_dev, kept_idx_dev, n_cache, ctx->status_dev);
    return launch_status(ctx, 1);
  }
  if (sh.maxN <= mkv::kSelectRegKeys) {                  // every segment fits the register-resident kernel
    // one wave of clusters (4 CTAs each, one CTA per SM): the leaner-latency variant; more segments: two CTAs per SM
    const bool one_wave = (long long)sh.R * sh.Hkv * mkv::kSelectCluster <= ctx->sm_count;
    mkv::launch_overlapped(one_wave ? mkv::select_kernel_reg<1> : mkv::select_kernel_reg<2>, dim3(sh.R * sh.Hkv * mkv::kSelectCluster),
                           dim3(mkv::kSelectRegThreads), (size_t)mkv::kSelectCandCap * 4, static_cast<cudaStream_t>(stream), sh, scores_dev,
                           budgets_dev, offsets_dev, kept_idx_dev, ctx->status_dev);
    return launch_status(ctx, 1);
  }
  const int max_cache = (ctx->smem_optin - mkv::kSelectStaticSmem) / 4;
  const int cache = sh.maxN <= max_cache ? sh.maxN : 0;   // segments that do not fit are read through L2
  mkv::select_kernel<<<sh.R * sh.Hkv, mkv::kSelectThreads, (size_t)cache * 4, static_cast<cudaStream_t>(stream)>>>(
      sh, scores_dev, budgets_dev, offsets_dev, kept_idx_dev, cache, ctx->status_dev);
  return launch_status(ctx, 1);
}

int maskkv_compact(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* k_prompt_dev, const void* v_prompt_dev,
                   const int32_t* kept_idx_dev, const int32_t* offsets_dev, int64_t capacity, void* kc_dev, void* vc_dev,
                   void* stream) {
  TraceRange trace("maskkv_compact");
  if (ctx == nullptr) return MASKKV_E_INVALID;
  Shape sh;
  int rc = resolve(desc, &sh);
  if (rc != MASKKV_OK) return rc;
  if (kept_idx_dev == nullptr || offsets_dev == nullptr || capacity < 0) return MASKKV_E_INVALID;
  if (capacity == 0 || sh.sumN == 0) return MASKKV_OK;
  if (k_prompt_dev == nullptr || v_prompt_dev == nullptr || kc_dev == nullptr || vc_dev == nullptr) return MASKKV_E_INVALID;
  if (!aligned16(k_prompt_dev) || !aligned16(v_prompt_dev) || !aligned16(kc_dev) || !aligned16(vc_dev)) return MASKKV_E_ALIGN;
  DeviceGuard guard(ctx->device);
  const int es = elem_size(sh.dtype);
  const long long warps = (capacity + mkv::kCompactRows - 1) / mkv::kCompactRows;
  long long blocks = (warps + (mkv::kCompactThreads / 32) - 1) / (mkv::kCompactThreads / 32);
  const long long max_blocks = (long long)ctx->sm_count * mkv::kCompactBlocksPerSm;
  if (blocks > max_blocks) blocks = max_blocks;
  auto kernel = 2 * sh.d * es / 16 <= 32 ? mkv::compact_kernel<1> : mkv::compact_kernel<2>;
  mkv::launch_overlapped(kernel, dim3((unsigned)blocks), dim3(mkv::kCompactThreads), 0, static_cast<cudaStream_t>(stream),
                         sh, sh.d * es, sh.kv_ts * es, sh.kv_hs * es, static_cast<const unsigned char*>(k_prompt_dev),
                         static_cast<const unsigned char*>(v_prompt_dev), kept_idx_dev, offsets_dev, (long long)capacity,
                         static_cast<unsigned char*>(kc_dev), static_cast<unsigned char*>(vc_dev), ctx->status_dev);
  return launch_status(ctx, 1);
}

int maskkv_attend(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* q_live_dev, const void* k_live_dev,
                  const void* v_live_dev, const void* kc_dev, const void* vc_dev, const int32_t* offsets_dev,
                  int64_t capacity, void* out_dev, float* lse_dev, void* stream) {
  return maskkv_attend_rows(ctx, desc, q_live_dev, nullptr, nullptr, k_live_dev, v_live_dev, kc_dev, vc_dev, offsets_dev, capacity,
                            out_dev, lse_dev, stream);
}

int maskkv_attend_rows(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* q_rows_dev, const int32_t* rows_cu,
                       const int32_t* rows_cu_dev, const void* k_live_dev, const void* v_live_dev, const void* kc_dev,
                       const void* vc_dev, const int32_t* offsets_dev, int64_t capacity, void* out_rows_dev, float* lse_rows_dev,
                       void* stream) {
  TraceRange trace("maskkv_attend_rows");
  if (ctx == nullptr) return MASKKV_E_INVALID;
  Shape sh;
  int rc = resolve(desc, &sh);
  if (rc != MASKKV_OK) return rc;
  if (offsets_dev == nullptr || capacity < 0) return MASKKV_E_INVALID;
  if ((rows_cu == nullptr) != (rows_cu_dev == nullptr)) return MASKKV_E_INVALID;
  // the query rows: the live rows themselves, or the caller's subset of them
  const int32_t* q_cu = sh.live_cu;
  int sum_q = sh.sumM, max_q = sh.maxM;
  if (rows_cu != nullptr) {
    if (rows_cu[0] != 0 || (reinterpret_cast<uintptr_t>(rows_cu_dev) & 3u)) return rows_cu[0] != 0 ? MASKKV_E_INVALID : MASKKV_E_ALIGN;
    max_q = 0;
    for (int r = 0; r < sh.R; ++r) {
      const long long n = (long long)rows_cu[r + 1] - rows_cu[r];
      if (n < 0) return MASKKV_E_INVALID;
      if (n > max_q) max_q = (int)n;
    }
    q_cu = rows_cu_dev;
    sum_q = rows_cu[sh.R];
  }
  if (sum_q == 0) return MASKKV_OK;
  if (q_rows_dev == nullptr || out_rows_dev == nullptr) return MASKKV_E_INVALID;
  if (sh.sumM > 0 && (k_live_dev == nullptr || v_live_dev == nullptr)) return MASKKV_E_INVALID;
  if (!aligned16(q_rows_dev) || !aligned16(k_live_dev) || !aligned16(v_live_dev) || !aligned16(kc_dev) ||
      !aligned16(vc_dev) || !aligned16(out_rows_dev))
    return MASKKV_E_ALIGN;
  DeviceGuard guard(ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (mkv::tc::attend_tc_supported(ctx, sh) && !(ctx->force_simt & 4u)) {
    if (mkv::tc::launch_attend_tc(ctx, sh, q_rows_dev, q_cu, sum_q, max_q, k_live_dev, v_live_dev, kc_dev, vc_dev, capacity, offsets_dev,
                                  out_rows_dev, lse_rows_dev, st) == 0) {
      ++ctx->tc_launches;
      return launch_status(ctx, 1);
    }
    ctx->host_flags |= MASKKV_FLAG_FALLBACK;               // the FP32-pipe kernel below takes over; nobody asked for it
  }
#define MKV_ATTEND(T, D) launch_attend_simt<T, D>(ctx, sh, q_rows_dev, q_cu, sum_q, max_q, k_live_dev, v_live_dev, kc_dev, vc_dev, \
                                                  offsets_dev, (long long)capacity, out_rows_dev, lse_rows_dev, st)
  if (sh.dtype == MASKKV_F32) return sh.d == 64 ? MKV_ATTEND(float, 64) : MKV_ATTEND(float, 128);
  return sh.d == 64 ? MKV_ATTEND(__nv_bfloat16, 64) : MKV_ATTEND(__nv_bfloat16, 128);
#undef MKV_ATTEND
}

#pragma GCC visibility pop
}  // extern "C"

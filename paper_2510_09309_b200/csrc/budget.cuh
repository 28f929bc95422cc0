// Head budgets (Eq. 14-15), clamp, capacity clip and the exclusive prefix sum that lays out the
// ragged cache.  One block; latency-bound by design (at most a few thousand segments).
//
// The floating-point part is IEEE double with explicit round-to-nearest intrinsics so that the
// compiler cannot contract a multiply and an add: the same fp32 masses give the same integers as any
// other IEEE implementation that evaluates the formula in the same order.
#pragma once

#include "common.cuh"

namespace mkv {

constexpr int kBudgetThreads = 256;
constexpr int kBudgetMaxSegments = 4096;

__device__ __forceinline__ double prompt_preference(float sp, float sm) {
  const double a = (double)sp, b = (double)sm;
  return __ddiv_rn(a, __dadd_rn(a, b));                 // Eq. 14
}

// dynamic shared memory: double P[S] | double T[R] | int k[S]
__global__ void __launch_bounds__(kBudgetThreads)
budget_kernel(Shape sh, int k_l, const int32_t* __restrict__ k_l_req, double alpha, double one_minus_alpha,
              const float* __restrict__ mass_p, const float* __restrict__ mass_m, long long capacity,
              int32_t* __restrict__ budgets, int32_t* __restrict__ offsets, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int S = sh.R * sh.Hkv;
  double* P = reinterpret_cast<double*>(smem_raw);
  double* T = P + S;
  int* kbuf = reinterpret_cast<int*>(T + sh.R);
  __shared__ long long warp_tot[kBudgetThreads / 32];
  const int tid = threadIdx.x;
  pdl_launch_dependents();
  pdl_wait();

  // the divisions are the slow part (double precision): all of them in parallel, then the sums in fixed order
  for (int s = tid; s < S; s += kBudgetThreads) P[s] = prompt_preference(mass_p[s], mass_m[s]);
  __syncthreads();
  for (int r = tid; r < sh.R; r += kBudgetThreads) {   // sum of preferences, ascending head order
    double t = 0.0;
    for (int h = 0; h < sh.Hkv; ++h) t = __dadd_rn(t, P[r * sh.Hkv + h]);
    T[r] = t;
  }
  __syncthreads();
  for (int s = tid; s < S; s += kBudgetThreads) {
    const int r = s / sh.Hkv;
    const int kl = k_l_req ? k_l_req[r] : k_l;
    const int n_r = sh.prompt_cu[r + 1] - sh.prompt_cu[r];
    const double phat = __ddiv_rn(P[s], T[r]);
    const double x = __dadd_rn(__dmul_rn(alpha, (double)kl),
                               __dmul_rn(__dmul_rn(one_minus_alpha, (double)((long long)sh.Hkv * kl)), phat));  // Eq. 15
    long long k = 0;
    if (x == x && fabs(x) < 1e18) k = (long long)floor(__dadd_rn(x, 1e-6));
    k = k < 0 ? 0 : (k > n_r ? n_r : k);
    kbuf[s] = (int)k;
  }
  __syncthreads();

  // exclusive scan: each thread owns a contiguous run of segments
  const int per = (S + kBudgetThreads - 1) / kBudgetThreads;
  const int b = min(tid * per, S), e = min(b + per, S);
  long long local = 0;
  for (int s = b; s < e; ++s) local += kbuf[s];
  long long incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long v = __shfl_up_sync(0xffffffffu, incl, o);
    if ((tid & 31) >= o) incl += v;
  }
  if ((tid & 31) == 31) warp_tot[tid >> 5] = incl;
  __syncthreads();
  long long base = 0;
  for (int w2 = 0; w2 < (tid >> 5); ++w2) base += warp_tot[w2];
  long long run = base + incl - local;
  bool clipped = false;
  for (int s = b; s < e; ++s) {
    const long long start = run < capacity ? run : capacity;
    const long long stop = run + kbuf[s] < capacity ? run + kbuf[s] : capacity;
    if (stop - start != kbuf[s]) clipped = true;
    run += kbuf[s];
    budgets[s] = (int)(stop - start);
    offsets[s] = (int)start;
    if (s == S - 1) offsets[S] = (int)stop;
  }
  if (clipped) atomicOr(status, (uint32_t)MASKKV_FLAG_CAPACITY);
}

}  // namespace mkv

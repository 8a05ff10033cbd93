// Per-layer figures of the last round, computed on request (lqsgd_step_stats): how many factor
// entries sat within one fp32 step of a decision threshold of the quantiser (Eq. 4), and how well
// conditioned the factor handed to Orthonormalize was (the Orthonormalize step of Algorithm 1).  Off the
// round's path: the kernel reads what the round left in the workspace (the orthonormal P, M Q
// before Orthonormalize, M^T P_bar, the scales) and writes three words per layer.
//
// "Within one step of a threshold": the quantiser decides on t = |x| / s, an fp32 number.  An
// entry counts when the fp32 neighbours of t on either side fall into different levels, i.e. a
// threshold b satisfies  below(t) < b <= above(t).  These are the entries whose code an
// implementation that forms |x| / s with a last-place difference may legitimately see differently.
//
// Pivot ratio: with M Q = P R (R upper triangular, positive diagonal) R_jj = P[:, j] . (M Q)[:, j];
// the figure is min_j R_jj / max_j R_jj, the smallest over the workers; 0 when a column was dropped.
#include "lqsgd_stats.h"

#include <math.h>

namespace lqsgd {

namespace {

constexpr int kStatsThreads = 256;

__device__ __forceinline__ int level_count(float t, const float* thr, int nthr) {
  int k = 0;
  for (int i = 0; i < nthr; ++i) k += (t >= thr[i]) ? 1 : 0;
  return k;
}

// 1 when the two fp32 neighbours of t = |x| / s lie in different levels.
__device__ __forceinline__ int near_threshold(float x, float s, const float* thr, int nthr) {
  const float t = __fdiv_rn(fabsf(x), s);
  if (!(t < INFINITY)) return 0;
  const float lo = t > 0.f ? __uint_as_float(__float_as_uint(t) - 1u) : 0.f;
  const float hi = __uint_as_float(__float_as_uint(t) + 1u);
  return level_count(lo, thr, nthr) != level_count(hi, thr, nthr) ? 1 : 0;
}

__device__ unsigned long long block_sum(unsigned long long v, unsigned long long* sh) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  unsigned long long tot = 0;
  if (threadIdx.x == 0)
    for (int i = 0; i < kStatsThreads / 32; ++i) tot += sh[i];
  return tot;            // valid on thread 0
}

// One CTA per (matrix layer, worker).
__global__ void __launch_bounds__(kStatsThreads) stats_kernel(StatsArgs a) {
  __shared__ float thr[2][128];
  __shared__ unsigned long long red[kStatsThreads / 32];
  __shared__ double diag[kMaxRank];
  __shared__ double part[kStatsThreads / 32];
  const LayerDev L = a.layers[blockIdx.x];
  const int w = blockIdx.y, RP = a.RP, r = L.r, tid = threadIdx.x;
  for (int i = tid; i < a.nthr_p; i += kStatsThreads) thr[0][i] = a.thr_p[i];
  for (int i = tid; i < a.nthr_q; i += kStatsThreads) thr[1][i] = a.thr_q[i];
  __syncthreads();

  for (int which = 0; which < 2; ++which) {
    const int rows = which ? L.m : L.n;
    const int nthr = which ? a.nthr_q : a.nthr_p;
    const float* x = (which ? L.Qw : L.P) + (size_t)w * rows * RP;
    unsigned long long near = 0;
    if (nthr > 0) {
      const long long count = (long long)rows * r;
      for (long long e = tid; e < count; e += kStatsThreads) {
        const int row = (int)(e / r), col = (int)(e - (long long)row * r);
        const float s = a.column_scales ? L.scales[which * RP + col] : L.scales[which];
        if (s > 0.f && s < INFINITY) near += near_threshold(x[(size_t)row * RP + col], s, thr[which], nthr);
      }
    }
    const unsigned long long tot = block_sum(near, red);
    if (tid == 0 && tot) atomicAdd(a.out + 4 * (size_t)blockIdx.x + which, tot);
  }

  // R_jj = sum_i P[i][j] (M Q)[i][j], in fp64; a thread takes rows tid, tid + 256, ... of one column at a time
  const float* P = L.P + (size_t)w * L.n * RP;
  const float* Praw = L.Praw + (size_t)w * L.n * RP;
  for (int j = 0; j < r; ++j) {
    double acc = 0.0;
    for (int i = tid; i < L.n; i += kStatsThreads) acc += (double)P[(size_t)i * RP + j] * (double)Praw[(size_t)i * RP + j];
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
    if ((tid & 31) == 0) part[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {                       // the warps' sums in warp order: the same bits every time
      double d = 0.0;
      for (int i = 0; i < kStatsThreads / 32; ++i) d += part[i];
      diag[j] = d;
    }
    __syncthreads();
  }
  if (tid == 0) {
    double lo = INFINITY, hi = 0.0;
    for (int j = 0; j < r; ++j) {
      const double d = diag[j] > 0.0 ? diag[j] : 0.0;
      lo = fmin(lo, d);
      hi = fmax(hi, d);
    }
    const float ratio = hi > 0.0 ? (float)(lo / hi) : 0.f;
    // non-negative floats order like their bit patterns: the smallest ratio over the workers
    atomicMin(reinterpret_cast<unsigned int*>(a.out + 4 * (size_t)blockIdx.x + 2), __float_as_uint(ratio));
  }
}

}  // namespace

cudaError_t launch_stats(const StatsArgs& a, int n_mat, cudaStream_t st) {
  if (n_mat == 0) return cudaSuccess;
  stats_kernel<<<dim3(n_mat, a.W), kStatsThreads, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace lqsgd

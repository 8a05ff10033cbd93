// The small steps of the LQ-SGD round between its streaming passes, as device functions:
//   Orthonormalize (Alg. 1) as CholeskyQR with the r x r part in fp64,
//   the factor exchange (Alg. 1: LogQuantize, All-Reduce, LogDequantize; Eq. 4, Eq. 1, Eq. 5),
//   the fixed-order reduction of pass 2's partial sums, the mean of the 1-D tensors.
// Each body does the work of one table entry ("job") with the threads of one CTA.  Two callers:
// the kernels of lqsgd_kernels.cu, one CTA per job, and the one-launch round of lqsgd_resident.cu,
// whose CTAs walk the same tables between grid barriers.
//
// Conventions.  NT threads take part (tid = 0 .. NT-1, every one of them calls the body and meets
// its __syncthreads()).  COH says where the inputs come from: false = an earlier kernel wrote them
// (read-only path), true = other CTAs of the SAME kernel wrote them before a grid barrier, so the
// loads must come from L2 (ld.global.cg), never from a line L1 may still hold.  `smem` is scratch
// of at least the body's ...Smem struct, 16-byte aligned; contents are dead on entry and exit
// (callers put a barrier between two jobs).
#pragma once
#include "lqsgd_dev.h"

#include <cuda_bf16.h>
#include <math.h>

namespace lqsgd {
namespace {

template <bool COH>
__device__ __forceinline__ float ld_in(const float* p) { return COH ? __ldcg(p) : __ldg(p); }
template <bool COH>
__device__ __forceinline__ double ld_in(const double* p) { return COH ? __ldcg(p) : __ldg(p); }

// N contiguous floats, aligned to min(N, 4) * 4 bytes
template <int N, bool COH>
__device__ __forceinline__ void load_contig(const float* __restrict__ p, float (&out)[N]) {
  if constexpr (N % 4 == 0) {
#pragma unroll
    for (int i = 0; i < N / 4; ++i) {
      const float4 v = COH ? __ldcg(reinterpret_cast<const float4*>(p) + i) : __ldg(reinterpret_cast<const float4*>(p) + i);
      out[4 * i] = v.x; out[4 * i + 1] = v.y; out[4 * i + 2] = v.z; out[4 * i + 3] = v.w;
    }
  } else if constexpr (N == 2) {
    const float2 v = COH ? __ldcg(reinterpret_cast<const float2*>(p)) : __ldg(reinterpret_cast<const float2*>(p));
    out[0] = v.x; out[1] = v.y;
  } else {
#pragma unroll
    for (int i = 0; i < N; ++i) out[i] = ld_in<COH>(p + i);
  }
}

template <int N>
__device__ __forceinline__ void store_contig(float* p, const float (&v)[N]) {
  if constexpr (N % 4 == 0) {
#pragma unroll
    for (int i = 0; i < N / 4; ++i)
      reinterpret_cast<float4*>(p)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
  } else if constexpr (N == 2) {
    *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]);
  } else {
#pragma unroll
    for (int i = 0; i < N; ++i) p[i] = v[i];
  }
}

// ---------------------------------------------------------------------------------------
// Orthonormalize (Alg. 1) as CholeskyQR with the r x r part in fp64:
//   p_reduce_gram: P_raw = sum of the column-chunk partials (fixed order); per-block Gram
//   p_apply      : Gram = sum of block Grams; R^T R = Gram; R^-1 (redone by every CTA);
//                  P = P_raw R^-1 (fp64 accumulate, stored fp32); block max |P|
// The result is the thin-QR Q factor with positive-diagonal R, the same matrix Gram-Schmidt
// produces.  A column whose pivot is <= 1e-10 of its squared norm (or zero, or not a number)
// becomes a zero column and the layer's status word says so.
// ---------------------------------------------------------------------------------------
constexpr double kPivotEps = 1e-10;

template <int RP> struct ReduceGramSmem {
  static constexpr int NSEG = RP <= 4 ? 8 : (RP == 8 ? 4 : 1);   // up to rank 8 an entry is summed in NSEG segments of the block's rows
  alignas(16) float rows[kFactorBlockRows][RP];                  // the block's rows (fp32: they are fp32 data)
  double seg[RP <= 8 ? NSEG : 1][RP <= 8 ? RP * RP : 1];
};

template <int RP, int NT, bool COH>
__device__ __forceinline__ void p_reduce_gram_body(const Tables& t, const FactorBlock fb, int tid, void* smem,
                                                   const LayerDev* staged = nullptr) {
  auto& S = *static_cast<ReduceGramSmem<RP>*>(smem);
  const LayerDev& L = staged ? *staged : t.layers[fb.layer];   // staged: the wrapper's copy of the entry
  const int n = L.n;
  if (tid < kFactorBlockRows) {
    const int row = fb.blk * kFactorBlockRows + tid;
    float p[RP];
#pragma unroll
    for (int j = 0; j < RP; ++j) p[j] = 0.f;
    if (row < n) {
      const float* src = L.Psum + ((size_t)fb.worker * L.nps * n + row) * RP;
      // the partials' loads go out together (8 at a time); the additions keep the chunk order
      int cc = 0;
      if constexpr (RP <= 8) {
        for (; cc + 8 <= L.nps; cc += 8) {
          float v[8][RP];
#pragma unroll
          for (int u = 0; u < 8; ++u) load_contig<RP, COH>(src + (size_t)(cc + u) * n * RP, v[u]);
#pragma unroll
          for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int j = 0; j < RP; ++j) p[j] += v[u][j];
        }
      }
      for (; cc < L.nps; ++cc) {
        float v[RP];
        load_contig<RP, COH>(src + (size_t)cc * n * RP, v);
#pragma unroll
        for (int j = 0; j < RP; ++j) p[j] += v[j];
      }
      if (L.ncc > 1) store_contig<RP>(L.Praw + ((size_t)fb.worker * n + row) * RP, p);
    }
#pragma unroll
    for (int j = 0; j < RP; ++j) S.rows[tid][j] = p[j];
  }
  __syncthreads();
  double* gp = L.gram_part + ((size_t)fb.worker * L.npb + fb.blk) * (RP * RP);
  if constexpr (RP >= 32) {
    // 4 x 4 entries per thread: two 128-bit reads of a row feed 16 multiply-adds (one entry per thread would read
    // two values per multiply-add, and the shared-memory reads, not the fp64 units, would set the pace)
    constexpr int TD = RP / 4;
    for (int tile = tid; tile < TD * TD; tile += NT) {
      const int ti = tile / TD, tj = tile % TD;
      if (tj < ti) continue;                               // symmetric: upper triangle of tiles, mirrored
      double acc[4][4];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
      for (int k = 0; k < kFactorBlockRows; ++k) {
        const float4 x = *reinterpret_cast<const float4*>(&S.rows[k][4 * ti]);
        const float4 y = *reinterpret_cast<const float4*>(&S.rows[k][4 * tj]);
        const double xa[4] = {(double)x.x, (double)x.y, (double)x.z, (double)x.w};
        const double yb[4] = {(double)y.x, (double)y.y, (double)y.z, (double)y.w};
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) acc[a][b] = fma(xa[a], yb[b], acc[a][b]);
      }
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          gp[(4 * ti + a) * RP + 4 * tj + b] = acc[a][b];
          gp[(4 * tj + b) * RP + 4 * ti + a] = acc[a][b];
        }
    }
  } else if constexpr (RP <= 8) {
    // few entries (at most 36 of the upper triangle): one thread per entry would leave the CTA idle behind a chain of
    // 128 dependent fp64 multiply-adds.  Every entry is summed over NSEG segments of the rows by NSEG threads, and the
    // segments' sums are added in segment order (the same split whatever the block size: the same bits on every path).
    constexpr int NE = RP * RP, NSEG = ReduceGramSmem<RP>::NSEG, SEG = kFactorBlockRows / NSEG;
    static_assert(NT >= NSEG * NE && kFactorBlockRows % NSEG == 0, "one thread per entry and segment");
    if (tid < NSEG * NE) {
      const int e = tid % NE, g = tid / NE, i = e / RP, j = e % RP;
      if (j >= i) {                                        // the Gram matrix is symmetric: upper triangle, mirrored
        double s = 0.0;
        for (int k = g * SEG; k < (g + 1) * SEG; ++k) s = fma((double)S.rows[k][i], (double)S.rows[k][j], s);
        S.seg[g][e] = s;
      }
    }
    __syncthreads();
    if (tid < NE) {
      const int i = tid / RP, j = tid % RP;
      if (j >= i) {
        double s = S.seg[0][tid];
#pragma unroll
        for (int g = 1; g < NSEG; ++g) s += S.seg[g][tid];
        gp[i * RP + j] = s;
        gp[j * RP + i] = s;
      }
    }
  } else {
    for (int e = tid; e < RP * RP; e += NT) {
      const int i = e / RP, j = e % RP;
      if (j < i) continue;                                 // the Gram matrix is symmetric: upper triangle, mirrored
      double s = 0.0;
      for (int k = 0; k < kFactorBlockRows; ++k) s = fma((double)S.rows[k][i], (double)S.rows[k][j], s);
      gp[i * RP + j] = s;
      gp[j * RP + i] = s;
    }
  }
}

// Cholesky of the Gram matrix in A (shared, complete and visible to the CTA on entry):  Gram = L L^T  (R = L^T).
// On return the lower triangle of A holds L, invd the reciprocals of its diagonal, dead[j] = 1 for a column
// dropped as dependent (its row and column of L are then those of the identity).  Returns true if any column
// was dropped.
template <int RP, int NT>
__device__ __forceinline__ bool cholesky_factor(double (*A)[RP + 1], double* diag0, int r, double* invd, int* dead, int tid) {
  if (tid < RP) { diag0[tid] = A[tid][tid]; dead[tid] = 0; invd[tid] = 1.0; }
  __syncthreads();
  // right-looking Cholesky by ONE warp (warp-level barriers only; the other warps wait once, below):
  // pivot, column j, then the rank-1 update of the trailing lower triangle with its entries dealt to
  // the lanes (every entry sees the updates in the order of j, so the result does not depend on how
  // the entries are dealt)
  if (tid < 32) {
    for (int j = 0; j < r; ++j) {
      const double d = A[j][j];
      const bool ok = (d > kPivotEps * diag0[j]) && (d < INFINITY);   // false for nan too
      // 1 / sqrt(d) by the hardware seed plus refinement (the library sqrt and division are long
      // software sequences, and this loop is a chain of r of them); l_jj = d / sqrt(d)
      const double inv = ok ? rsqrt(d) : 1.0;
      const double ljj = ok ? d * inv : 1.0;
      __syncwarp();                      // every lane has read the pivot
      for (int i = j + tid; i < r; i += 32) {
        if (i == j) { A[j][j] = ljj; invd[j] = inv; if (!ok) dead[j] = 1; }
        else A[i][j] = ok ? A[i][j] * inv : 0.0;
      }
      __syncwarp();
      if (ok) {
        const int w = r - j - 1;         // trailing block: rows and columns j+1 .. r-1
        for (int e = tid; e < w * w; e += 32) {
          const int i = j + 1 + e / w, k = j + 1 + e % w;
          if (k <= i) A[i][k] -= A[i][j] * A[k][j];
        }
      }
      __syncwarp();
    }
  }
  __syncthreads();
  int any = 0;
  for (int j = 0; j < r; ++j) any |= dead[j];
  return any != 0;
}

// Gram = sum of the block Grams (block order), then its Cholesky factor, by a whole CTA; every CTA that
// orthonormalises a block of rows redoes this small factorisation itself, which costs less than a
// kernel boundary.
template <int RP> struct CholSmem {
  static constexpr int SEG = (RP * RP <= 64) ? 128 / (RP * RP) : 1;   // at least 128 threads take part
  double A[RP][RP + 1];                // Gram, overwritten by L (lower triangle)
  double segsum[SEG > 1 ? SEG : 1][SEG > 1 ? RP * RP : 1];
  double diag0[RP];
};

template <int RP, int NT, bool COH>
__device__ __forceinline__ bool cholesky_lower(const LayerDev& L, int worker, CholSmem<RP>& C, double* invd, int* dead, int tid) {
  // Gram = sum of the block Grams.  With more threads than entries the blocks are dealt to SEG
  // segments (segment g takes blocks g, g + SEG, ...), eight loads in flight each; the segments'
  // sums are then added in segment order: a fixed order, and a chain SEG times shorter.
  constexpr int SEG = CholSmem<RP>::SEG;
  if constexpr (SEG > 1) {
    if (tid < SEG * RP * RP) {
      const int e = tid % (RP * RP), g = tid / (RP * RP);
      const double* gp = L.gram_sum + (size_t)worker * L.ngs * (RP * RP) + e;
      double s = 0.0;
      int b = g;
      for (; b + 7 * SEG < L.ngs; b += 8 * SEG) {
        double x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = ld_in<COH>(gp + (size_t)(b + u * SEG) * (RP * RP));
#pragma unroll
        for (int u = 0; u < 8; ++u) s += x[u];
      }
      for (; b < L.ngs; b += SEG) s += ld_in<COH>(gp + (size_t)b * (RP * RP));
      C.segsum[g][e] = s;
    }
    __syncthreads();
    if (tid < RP * RP) {
      double s = C.segsum[0][tid];
#pragma unroll
      for (int g = 1; g < SEG; ++g) s += C.segsum[g][tid];
      C.A[tid / RP][tid % RP] = s;
    }
  } else {
    for (int e = tid; e < RP * RP; e += NT) {
      const double* gp = L.gram_sum + (size_t)worker * L.ngs * (RP * RP) + e;
      double s = 0.0;
      int b = 0;
      for (; b + 8 <= L.ngs; b += 8) {        // eight loads in flight, additions in block order
        double x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = ld_in<COH>(gp + (size_t)(b + u) * (RP * RP));
#pragma unroll
        for (int u = 0; u < 8; ++u) s += x[u];
      }
      for (; b < L.ngs; ++b) s += ld_in<COH>(gp + (size_t)b * (RP * RP));
      C.A[e / RP][e % RP] = s;
    }
  }
  __syncthreads();
  return cholesky_factor<RP, NT>(C.A, C.diag0, L.r, invd, dead, tid);
}

// Padded rank >= kCholSplitRP: Gram = sum of the block Grams and its Cholesky factor, ONCE per (layer, worker), by a CTA
// of its own whose threads all take part in the trailing updates (CTA barriers between the steps); the factor,
// the reciprocals of its diagonal and the dropped-column flags go to L.chol for p_apply_body to fetch.
template <int RP, int NT> struct CholOnceSmem {
  double A[RP][RP + 1];
  double diag0[RP];
  double invd[RP];
  int dead[RP];
};

template <int RP, int NT, bool COH>
__device__ __forceinline__ void p_chol_body(const Tables& t, const FactorBlock fb, int tid, void* smem,
                                            const LayerDev* staged = nullptr) {
  auto& S = *static_cast<CholOnceSmem<RP, NT>*>(smem);
  const LayerDev& L = staged ? *staged : t.layers[fb.layer];   // staged: the wrapper's copy of the entry
  const int r = L.r;
  for (int e = tid; e < RP * RP; e += NT) {
    const double* gp = L.gram_sum + (size_t)fb.worker * L.ngs * (RP * RP) + e;
    double s = 0.0;
    int b = 0;
    for (; b + 8 <= L.ngs; b += 8) {        // eight loads in flight, additions in block order
      double x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) x[u] = ld_in<COH>(gp + (size_t)(b + u) * (RP * RP));
#pragma unroll
      for (int u = 0; u < 8; ++u) s += x[u];
    }
    for (; b < L.ngs; ++b) s += ld_in<COH>(gp + (size_t)b * (RP * RP));
    S.A[e / RP][e % RP] = s;
  }
  __syncthreads();
  if (tid < RP) { S.diag0[tid] = S.A[tid][tid]; S.dead[tid] = 0; S.invd[tid] = 1.0; }
  // Right-looking, ONE barrier per step: column j stays unscaled while the steps run (the update of entry (i, k)
  // takes a_ij a_kj (1 / sqrt d_j)^2 instead of (a_ij / sqrt d_j)(a_kj / sqrt d_j)); the columns are scaled at the end.  The
  // threads form a 16 x 16 grid over the trailing block's rows and columns (no index arithmetic with divisions).
  static_assert(NT == 256, "16 x 16 threads");
  const int ta = tid >> 4, tb = tid & 15;
  for (int j = 0; j < r; ++j) {
    __syncthreads();                       // the updates of step j - 1 (and the initial values) are in place
    const double d = S.A[j][j];
    const bool ok = (d > kPivotEps * S.diag0[j]) && (d < INFINITY);   // false for nan too
    const double inv = ok ? rsqrt(d) : 1.0;       // (hardware seed plus refinement: a division is a much longer sequence)
    if (tid == 0) { S.invd[j] = inv; if (!ok) S.dead[j] = 1; }
    if (ok) {
      const double inv2 = inv * inv;
      for (int i = j + 1 + ta; i < r; i += 16) {
        const double aij = S.A[i][j] * inv2;
        for (int k = j + 1 + tb; k <= i; k += 16) S.A[i][k] -= aij * S.A[k][j];
      }
    }
  }
  __syncthreads();
  // L: column j of the lower triangle times 1 / sqrt d_j; a dropped column is that of the identity
  for (int e = tid; e < r * RP; e += NT) {
    const int i = e / RP, j = e - i * RP;
    if (j < r && j <= i) {
      const bool deadj = S.dead[j] != 0;
      S.A[i][j] = (i == j) ? (deadj ? 1.0 : S.A[j][j] * S.invd[j]) : (deadj ? 0.0 : S.A[i][j] * S.invd[j]);
    }
  }
  __syncthreads();
  double* dst = L.chol + (size_t)fb.worker * (RP * RP + 2 * RP);
  for (int e = tid; e < RP * RP; e += NT) dst[e] = S.A[e / RP][e % RP];
  if (tid < RP) { dst[RP * RP + tid] = S.invd[tid]; dst[RP * RP + RP + tid] = S.dead[tid] ? 1.0 : 0.0; }
  if (tid == 0) {
    int any = 0;
    for (int j = 0; j < r; ++j) any |= S.dead[j];
    if (any) atomicOr(&t.status[fb.layer], 1u);
  }
}

template <int RP, int NT> struct ApplySmem {
  CholSmem<RP> chol;
  double invd[RP];
  int dead[RP];
  float smax[NT / 32];
  float scol[NT / 32][RP];
};

// One block of kFactorBlockRows rows of one worker's P: thread tid < kFactorBlockRows owns a row.
template <int RP, int NT, bool COH>
__device__ __forceinline__ void p_apply_body(const Tables& t, const FactorBlock fb, int tid, void* smem,
                                             const LayerDev* staged = nullptr) {
  static_assert(NT >= kFactorBlockRows, "one thread per row of the block");
  auto& S = *static_cast<ApplySmem<RP, NT>*>(smem);
  const LayerDev& L = staged ? *staged : t.layers[fb.layer];   // staged: the wrapper's copy of the entry
  const int n = L.n;
  if constexpr (RP >= kCholSplitRP) {
    // the factor was computed once for this (layer, worker) by p_chol_body: fetch it
    const double* src = L.chol + (size_t)fb.worker * (RP * RP + 2 * RP);
    for (int e = tid; e < RP * RP; e += NT) S.chol.A[e / RP][e % RP] = ld_in<COH>(src + e);
    if (tid < RP) { S.invd[tid] = ld_in<COH>(src + RP * RP + tid); S.dead[tid] = ld_in<COH>(src + RP * RP + RP + tid) != 0.0; }
    __syncthreads();
  } else {
    const bool dropped = cholesky_lower<RP, NT, COH>(L, fb.worker, S.chol, S.invd, S.dead, tid);
    if (dropped && fb.blk == 0 && tid == 0) atomicOr(&t.status[fb.layer], 1u);
  }
  if (L.qfused && fb.blk == 0)                 // the block maxima of |Q_w| that pass 2 will raise start from zero
    for (int i = tid; i < L.nqb; i += NT) L.maxq[(size_t)fb.worker * L.nqb + i] = 0.f;
  const int row = fb.blk * kFactorBlockRows + tid;
  float o[RP];
#pragma unroll
  for (int j = 0; j < RP; ++j) o[j] = 0.f;
  float amax = 0.f;
  if (tid < kFactorBlockRows && row < n) {
    // the row of P solves  o R = p  with R = L^T upper triangular: forward substitution in fp64,
    //   o[j] = (p[j] - sum_{k<j} o[k] L[j][k]) / L[j][j];   a dropped column gives 0
    float p[RP];
    load_contig<RP, COH>(L.Praw + ((size_t)fb.worker * n + row) * RP, p);
    // Column by column: once o[k] is known it is taken out of every later entry.  Each entry still sees its terms in
    // the order k = 0, 1, ... (the same sums, the same bits as entry by entry), but the updates of one k are
    // independent of one another, where the sum of one entry is a chain of dependent fp64 operations.
    double sd[RP];
#pragma unroll
    for (int j = 0; j < RP; ++j) sd[j] = (double)p[j];
    bool bad = false;
#pragma unroll
    for (int k = 0; k < RP; ++k) {
      const double ok_ = (k < L.r && !S.dead[k]) ? sd[k] * S.invd[k] : 0.0;
      o[k] = (float)ok_;
      amax = fmaxf(amax, fabsf(o[k]));
      bad |= !(fabsf(o[k]) < INFINITY);
#pragma unroll
      for (int j = k + 1; j < RP; ++j) sd[j] = fma(-ok_, S.chol.A[j][k], sd[j]);
    }
    store_contig<RP>(L.P + ((size_t)fb.worker * n + row) * RP, o);
    if (bad) atomicOr(&t.status[fb.layer], 8u);
  }
  if (t.col_scales) {            // variant: one maximum per column
#pragma unroll
    for (int j = 0; j < RP; ++j) {
      float v = fabsf(o[j]);
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
      if ((tid & 31) == 0) S.scol[tid >> 5][j] = v;
    }
    __syncthreads();
    if (tid < RP) {
      float a = S.scol[0][tid];
#pragma unroll
      for (int w = 1; w < NT / 32; ++w) a = fmaxf(a, S.scol[w][tid]);
      L.maxp[((size_t)fb.worker * L.npb + fb.blk) * RP + tid] = a;
    }
    return;
  }
  // max over the block; NaN compares false and is dropped (reported separately)
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
  if ((tid & 31) == 0) S.smax[tid >> 5] = amax;
  __syncthreads();
  if (tid == 0) {
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) amax = fmaxf(amax, S.smax[w]);
    L.maxp[(size_t)fb.worker * L.npb + fb.blk] = amax;
  }
}

// Orthonormalize for a layer of at most 512 rows (every layer of the ResNet-18 set), one CTA of 512 threads per
// (layer, worker), one thread per row: the sum of pass 1's column-chunk partials, the Gram matrix in
// fp64 (every entry summed over eight 64-row segments, the segments then added in order), its
// Cholesky factor, the rows of P by substitution and the block maxima: what p_reduce_gram and
// p_apply do in two steps for taller layers.
constexpr int kOrthSmallRows = 512;
template <int RP> struct OrthSmallSmem {
  static constexpr int NE = RP * RP, NSEG = 8;
  double rows[kOrthSmallRows][RP];
  double seg[NSEG][NE];
  double A[RP][RP + 1];
  double diag0[RP];
  double invd[RP];
  int dead[RP];
  float wmax[kOrthSmallRows / 32][RP];
};

template <int RP, bool COH>
__device__ __forceinline__ void p_orth_small_body(const Tables& t, const FactorBlock fb, int tid, void* smem,
                                                  const LayerDev* staged = nullptr) {
  using SM = OrthSmallSmem<RP>;
  constexpr int NE = SM::NE, NSEG = SM::NSEG, SEGROWS = kOrthSmallRows / NSEG;
  auto& S = *static_cast<SM*>(smem);
  const LayerDev& L = staged ? *staged : t.layers[fb.layer];   // staged: the wrapper's copy of the entry
  const int n = L.n, row = tid;
  float p[RP];
#pragma unroll
  for (int j = 0; j < RP; ++j) p[j] = 0.f;
  if (row < n) {
    const float* src = L.Psum + ((size_t)fb.worker * L.nps * n + row) * RP;
    for (int cc = 0; cc < L.nps; ++cc) {
      float v[RP];
      load_contig<RP, COH>(src + (size_t)cc * n * RP, v);
#pragma unroll
      for (int j = 0; j < RP; ++j) p[j] += v[j];
    }
    if (L.ncc > 1) store_contig<RP>(L.Praw + ((size_t)fb.worker * n + row) * RP, p);
  }
#pragma unroll
  for (int j = 0; j < RP; ++j) S.rows[tid][j] = (double)p[j];
  __syncthreads();
  for (int idx = tid; idx < NSEG * NE; idx += kOrthSmallRows) {
    const int e = idx % NE, g = idx / NE, i = e / RP, j = e % RP;
    if (j < i) continue;                                   // upper triangle; mirrored below
    double s = 0.0;
    for (int k = g * SEGROWS; k < (g + 1) * SEGROWS; ++k) s = fma(S.rows[k][i], S.rows[k][j], s);
    S.seg[g][e] = s;
  }
  __syncthreads();
  if (tid < NE) {
    const int i = tid / RP, j = tid % RP;
    if (j >= i) {
      double s = S.seg[0][tid];
#pragma unroll
      for (int g = 1; g < NSEG; ++g) s += S.seg[g][tid];
      S.A[i][j] = s;
      S.A[j][i] = s;
    }
  }
  __syncthreads();
  const bool dropped = cholesky_factor<RP, kOrthSmallRows>(S.A, S.diag0, L.r, S.invd, S.dead, tid);
  if (dropped && tid == 0) atomicOr(&t.status[fb.layer], 1u);
  float o[RP];
#pragma unroll
  for (int j = 0; j < RP; ++j) o[j] = 0.f;
  if (row < n) {
    double od[RP];
    bool bad = false;
#pragma unroll
    for (int j = 0; j < RP; ++j) {
      double s = (double)p[j];
#pragma unroll
      for (int k = 0; k < j; ++k) s = fma(-od[k], S.A[j][k], s);
      od[j] = (j < L.r && !S.dead[j]) ? s * S.invd[j] : 0.0;
      o[j] = (float)od[j];
      bad |= !(fabsf(o[j]) < INFINITY);
    }
    store_contig<RP>(L.P + ((size_t)fb.worker * n + row) * RP, o);
    if (bad) atomicOr(&t.status[fb.layer], 8u);
  }
  // maxima per block of 128 rows (4 warps), as the exchange reads them; one per column in the column-scale variant
#pragma unroll
  for (int j = 0; j < RP; ++j) {
    float v = fabsf(o[j]);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
    if ((tid & 31) == 0) S.wmax[tid >> 5][j] = v;
  }
  __syncthreads();
  const int ncs = t.col_scales ? RP : 1;
  if (tid < L.npb * ncs) {
    const int blk = tid / ncs, j0 = tid % ncs;
    float a = 0.f;
    for (int w4 = 4 * blk; w4 < 4 * blk + 4; ++w4)
      for (int j = (t.col_scales ? j0 : 0); j < (t.col_scales ? j0 + 1 : RP); ++j) a = fmaxf(a, S.wmax[w4][j]);
    L.maxp[((size_t)fb.worker * L.npb + blk) * ncs + j0] = a;
  }
}

// Q_w = sum of the row-chunk partials of pass 2, in chunk order; block max |Q_w|.  A thread owns
// V = min(RP, 4) consecutive columns of a row (one 128-bit load per partial when RP >= 4) and the
// loads of several partials are in flight together: the chain of nrb dependent additions, not a
// chain of nrb memory latencies, is what a row costs.
template <int RP, int NT> struct QReduceSmem {
  static constexpr int V = RP < 4 ? RP : 4, TPR = RP / V;
  float smax[NT / 32][TPR * V];
};

template <int RP, int NT, bool COH>
__device__ __forceinline__ void q_reduce_body(const Tables& t, const FactorBlock fb, int tid, void* smem,
                                              const LayerDev* staged = nullptr) {
  constexpr int V = RP < 4 ? RP : 4;        // floats per thread item
  constexpr int TPR = RP / V;               // items per row: 1, 2, 4 or 8 (divides the block size and 32)
  auto& S = *static_cast<QReduceSmem<RP, NT>*>(smem);
  const LayerDev& L = staged ? *staged : t.layers[fb.layer];   // staged: the wrapper's copy of the entry
  const int m = L.m, nrb = L.nqs;
  const size_t plane = (size_t)m * RP;      // floats of one partial
  float cmax[V];
#pragma unroll
  for (int v = 0; v < V; ++v) cmax[v] = 0.f;
  bool bad = false;
  for (int item = tid; item < kFactorBlockRows * TPR; item += NT) {
    const int row = fb.blk * kFactorBlockRows + item / TPR;
    if (row >= m) break;
    const size_t off = (size_t)row * RP + (size_t)(item % TPR) * V;
    const float* src = L.Qsum + (size_t)fb.worker * nrb * plane + off;
    float q[V];
#pragma unroll
    for (int v = 0; v < V; ++v) q[v] = 0.f;
    int rb = 0;
    for (; rb + 8 <= nrb; rb += 8) {
      float x[8][V];
#pragma unroll
      for (int u = 0; u < 8; ++u) load_contig<V, COH>(src + (size_t)(rb + u) * plane, x[u]);
#pragma unroll
      for (int u = 0; u < 8; ++u)
#pragma unroll
        for (int v = 0; v < V; ++v) q[v] += x[u][v];
    }
    for (; rb < nrb; ++rb) {
      float x[V];
      load_contig<V, COH>(src + (size_t)rb * plane, x);
#pragma unroll
      for (int v = 0; v < V; ++v) q[v] += x[v];
    }
    if (L.nrb > 1) store_contig<V>(L.Qw + (size_t)fb.worker * plane + off, q);
#pragma unroll
    for (int v = 0; v < V; ++v) {
      cmax[v] = fmaxf(cmax[v], fabsf(q[v]));
      bad |= !(fabsf(q[v]) < INFINITY);
    }
  }
  if (bad) atomicOr(&t.status[fb.layer], 8u);
  // maxima: the columns a thread owns are fixed (NT and 32 are multiples of TPR): columns (tid % TPR) V + v
  const int warp = tid >> 5, lane = tid & 31;
  if (t.col_scales) {
#pragma unroll
    for (int v = 0; v < V; ++v) {
#pragma unroll
      for (int o = 16; o >= TPR; o >>= 1) cmax[v] = fmaxf(cmax[v], __shfl_xor_sync(0xffffffffu, cmax[v], o));
      if (lane < TPR) S.smax[warp][lane * V + v] = cmax[v];
    }
    __syncthreads();
    if (tid < RP) {
      float a = S.smax[0][tid];
#pragma unroll
      for (int w = 1; w < NT / 32; ++w) a = fmaxf(a, S.smax[w][tid]);
      L.maxq[((size_t)fb.worker * L.nqb + fb.blk) * RP + tid] = a;
    }
    return;
  }
  float amax = cmax[0];
#pragma unroll
  for (int v = 1; v < V; ++v) amax = fmaxf(amax, cmax[v]);
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if (lane == 0) S.smax[warp][0] = amax;
  __syncthreads();
  if (tid == 0) {
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) amax = fmaxf(amax, S.smax[w][0]);
    L.maxq[(size_t)fb.worker * L.nqb + fb.blk] = amax;
  }
}

// One element of an averaged factor (P_bar or Q_bar) goes to its row-major home and to the
// copies the passes read: the transposed Q of passes 1 and 3 and, for layers on the tensor-core
// passes, the operands in the narrow terms those passes multiply (see lqsgd_tc.cu).
__device__ __forceinline__ float tf32_remainder(float x) {
  return x - __uint_as_float(__float_as_uint(x) & 0xffffe000u);
}
template <int RP>
__device__ __forceinline__ void store_factor(const LayerDev& L, int which, int row, int col, float v) {
  if (which) {
    L.Q[(size_t)row * RP + col] = v;
    L.Qt[(size_t)col * L.mt + row] = v;
    if (L.tc) {
      const float lo = tf32_remainder(v);
      L.Qt[(size_t)(RP + col) * L.mt + row] = lo;
      float* qc = L.Qcat + (size_t)row * L.kcat + col;
      qc[0] = v; qc[RP] = lo; qc[2 * RP] = v;
    }
  } else {
    L.Pbar[(size_t)row * RP + col] = v;
    if (L.tc) {
      float* pc = L.Pcat + (size_t)row * L.kcat + col;
      pc[0] = v; pc[RP] = v; pc[2 * RP] = tf32_remainder(v);
      // three bf16 terms v = b1 + b2 + b3 (24 bits), each stored twice in one word: the two K slots
      // that face the bf16 pair of an element of M in the tensor-core pass 2
      float rest = v;
#pragma unroll
      for (int term = 0; term < 3; ++term) {
        const __nv_bfloat16 b = __float2bfloat16_rn(rest);
        rest -= __bfloat162float(b);
        const uint32_t h = __bfloat16_as_ushort(b);
        reinterpret_cast<uint32_t*>(L.Pbt)[(size_t)(term * RP + col) * L.nt + row] = h | (h << 16);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// 1-D tensors: mean over the workers (Eq. 1) in worker order, and the raw fp32 values into
// each worker's payload.  One job = 256 entries of one tensor (threads tid < 256).
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void vectors_block(const VectorJob& vj, int job, int tid, uint8_t* payload, uint64_t payload_stride,
                                              int W) {
  const ExchangeChunk ch = vj.chunks[job];
  const VectorDev v = vj.vecs[ch.layer];
  const int i = ch.chunk * 256 + tid;
  if (tid >= 256 || i >= v.len) return;
  float s = 0.f;
  for (int w = 0; w < W; ++w) {
    const float x = vj.vgrads[(size_t)ch.layer * W + w][i];
    reinterpret_cast<float*>(payload + (size_t)w * payload_stride + v.pay_off)[i] = x;
    s += x;
  }
  const float mean = s / (float)vj.W_total;     // with workers on other GPUs too: this rank's share of the mean
  if (vj.xvec) { vj.xvec[(v.pay_off - vj.xvec_base) / 4 + i] = mean; return; }   // summed over the ranks before it is used
  if (vj.vghat[ch.layer]) vj.vghat[ch.layer][i] = mean;
  if (vj.vweights && vj.vweights[ch.layer]) vj.vweights[ch.layer][i] = fmaf(-vj.lr, mean, vj.vweights[ch.layer][i]);
}

// ---------------------------------------------------------------------------------------
// Factor exchange (Alg. 1: LogQuantize, All-Reduce, LogDequantize) for one chunk of 256
// factor elements of one layer, all W workers:
//   s      = max |x| over the layer's block maxima (shared scale)
//   code_w = sign bit | k,  k = number of thresholds <= |x_w| / s        (Eq. 4, nearest level)
//   stream = little-endian b-bit packing of code_w into worker w's payload
//   S      = sum_w (+-k_w)   exact integer;   x_bar = s * deq[S]          (Eq. 1, Eq. 5)
// The threshold table holds, for every level boundary, the smallest fp32 not below the exact
// boundary, so "t >= thr" decides exactly like the real-number comparison.
// B = bits per code (2..8), or 32: quantiser bypassed; B = 0: the bit count is read from qt.bits at run
// time (one instantiation for all bit counts, loops not unrolled).  Thread tid < 256 owns one element.
// ---------------------------------------------------------------------------------------
// Level index k (0 .. nlev - 1) of |x| at scale s: the number of thresholds <= |x| / s, by halving steps over
// the ascending table (nlev - 1 = 2^(b-1) - 1 entries in shared memory); |x| / s is an IEEE fp32 division.
__device__ __forceinline__ int level_of(float x, float s, const float* thr, int nlev) {
  const float tt = __fdiv_rn(fabsf(x), s);
  int k = 0;
  for (int step = nlev >> 1; step >= 1; step >>= 1)
    if (tt >= thr[k + step - 1]) k += step;
  return k;
}
// The same as a real call: the one-launch round runs every step once per launch, from a cold instruction
// cache, so there the size of the code counts for more than a call does.
__device__ __noinline__ int level_of_call(float x, float s, const float* thr, int nlev) { return level_of(x, s, thr, nlev); }

template <int RP, int NT> struct ExchangeSmem {
  float thr[128];
  alignas(4) uint8_t codes[8][kExchangeChunk + 4];
  float sred[NT / 32];
  float scol[RP];
};

// PLAIN: Algorithm 1's exchange as it stands - one scale per factor, average of the level indices, all workers on
// this GPU - with the variants compiled out: the kernel is then half the size, and for a step this short the
// size of its code is a large part of its cost.
template <int RP, int B, int NT, bool COH, bool PLAIN = false>
__device__ __forceinline__ void exchange_body(const Tables& t, const QuantTables& qt_in, int which, const ExchangeChunk ch,
                                              const SplitExchange& sx_in, int tid, void* smem,
                                              const LayerDev* staged = nullptr) {
  struct QtView { const float* thr; const float* deq; int32_t bits; int32_t avg_values; };
  struct SxView { int32_t pack_only, n_mat, ns; const float* scales; uint8_t* send[2]; uint64_t region_bytes[2], region_off[2]; };
  const QtView qt{qt_in.thr, qt_in.deq, qt_in.bits, PLAIN ? 0 : qt_in.avg_values};
  const SxView sx{PLAIN ? 0 : sx_in.pack_only, sx_in.n_mat, sx_in.ns, sx_in.scales, {sx_in.send[0], sx_in.send[1]},
                  {sx_in.region_bytes[0], sx_in.region_bytes[1]}, {sx_in.region_off[0], sx_in.region_off[1]}};
  constexpr int CH = kExchangeChunk;   // 256 factor elements per job, one per thread
  constexpr int WB = 8;                // workers handled per round
  const int bits = B ? B : qt.bits;    // a compile-time constant unless B == 0
  const int NLEV = (bits == 32) ? 2 : 1 << (bits - 1);
  static_assert(NT >= CH && NT % 32 == 0 && (NT % RP == 0), "block shape");
  auto& S = *static_cast<ExchangeSmem<RP, NT>*>(smem);
  const LayerDev& L = staged ? *staged : t.layers[ch.layer];
  const int W = t.W;
  const int rows = which ? L.m : L.n, r = L.r;
  const int count = rows * r;
  const int nblk = which ? L.nqb : L.npb;
  const float* __restrict__ maxes = which ? L.maxq : L.maxp;
  const float* __restrict__ src = which ? L.Qw : L.P;   // [W][rows][RP]
  const uint64_t pay_off = which ? L.pay_q_off : L.pay_p_off;

  // the first workers' values of this thread's element are on their way before the scale is known: the loads
  // do not depend on it, and what this job costs is its chain of dependent memory latencies
  float xfirst[WB];
  {
    const int e1 = ch.chunk * CH + tid;
    const bool v1 = tid < CH && e1 < count;
    const int row1 = v1 ? e1 / r : 0, col1 = v1 ? e1 % r : 0;
#pragma unroll
    for (int u = 0; u < WB; ++u)
      xfirst[u] = (v1 && u < W) ? ld_in<COH>(src + ((size_t)u * rows + row1) * RP + col1) : 0.f;
  }
  for (int i = tid; i < NLEV - 1; i += NT) S.thr[i] = qt.thr[i];
  // With at most 7 thresholds (b <= 4) a kernel of its own keeps them in registers and counts the thresholds not
  // above |x| / s directly (the same number the halving search finds in the ascending table): at ranks 16 and up
  // this kernel is bound by its instruction count, and the search with its call was half of it.
  constexpr bool kRegThr = !COH && B >= 2 && B <= 4;
  constexpr int kNThr = kRegThr ? (1 << (B - 1)) - 1 : 1;
  float thr_r[kNThr];
  if constexpr (kRegThr) {
#pragma unroll
    for (int i = 0; i < kNThr; ++i) thr_r[i] = __ldg(qt.thr + i);
  }
  if (tid < WB) *reinterpret_cast<uint32_t*>(&S.codes[tid][CH]) = 0u;     // what a word task reads past the chunk
  float s = 0.f;
  const bool cs = PLAIN ? false : t.col_scales != 0;
  if (cs) {
    // variant: one scale per column.  Block maxima are [W][nblk][RP]; thread tid only meets column tid % RP.
    // (a maximum of non-negative floats is the maximum of their bit patterns as integers: exact, in any order)
    if (tid < RP) S.scol[tid] = 0.f;
    __syncthreads();
    for (int i = tid; i < W * nblk * RP; i += NT) s = fmaxf(s, ld_in<COH>(maxes + i));
    atomicMax(reinterpret_cast<int*>(S.scol) + tid % RP, __float_as_int(s));
    __syncthreads();
    if (sx.pack_only) {                                   // scales agreed between the ranks
      if (tid < RP) S.scol[tid] = sx.scales[(size_t)(which * sx.n_mat + ch.layer) * sx.ns + tid];
      __syncthreads();
    }
  } else {
    for (int i = tid; i < W * nblk; i += NT) s = fmaxf(s, ld_in<COH>(maxes + i));
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) s = fmaxf(s, __shfl_xor_sync(0xffffffffu, s, o));
    if ((tid & 31) == 0) S.sred[tid >> 5] = s;
    __syncthreads();
    s = S.sred[0];
#pragma unroll
    for (int i = 1; i < NT / 32; ++i) s = fmaxf(s, S.sred[i]);
    if (sx.pack_only) s = sx.scales[(size_t)(which * sx.n_mat + ch.layer) * sx.ns];   // scale agreed between the ranks
  }
  // scales, status: once per layer
  if (ch.chunk == 0 && (cs ? tid < r : tid == 0)) {
    const float sj = cs ? S.scol[tid] : s;
    L.scales[cs ? which * RP + tid : which] = sj;
    for (int w = 0; w < W; ++w) {
      float* ps = reinterpret_cast<float*>(t.payload + (size_t)w * t.payload_stride + L.pay_scale_off);
      ps[cs ? which * r + tid : which] = sj;
    }
    if (bits != 32 && !(sj > 0.f)) atomicOr(&t.status[ch.layer], which ? 4u : 2u);
    if (!(sj < INFINITY)) atomicOr(&t.status[ch.layer], 8u);
  }

  if (bits == 32) {
    // Quantiser bypassed (plain PowerSGD exchange): the factor travels as fp32 and the workers'
    // factors are averaged directly (Eq. 1), in worker order.
    const int e = ch.chunk * CH + tid;
    if (tid < CH && e < count) {
      const int row = e / r, col = e - row * r;
      float sum = 0.f;
      for (int w = 0; w < W; ++w) {
        const float x = w < WB ? xfirst[w] : ld_in<COH>(src + ((size_t)w * rows + row) * RP + col);
        sum += x;
        uint8_t* pay = t.payload + (size_t)w * t.payload_stride + pay_off + (size_t)e * 4;
        const unsigned bits32 = __float_as_uint(x);               // the stream may start on any byte
        pay[0] = bits32 & 0xff; pay[1] = (bits32 >> 8) & 0xff; pay[2] = (bits32 >> 16) & 0xff; pay[3] = bits32 >> 24;
        if (sx.pack_only) {                                       // the same bytes, contiguous, for the all-gather
          uint8_t* snd = sx.send[which] + (size_t)w * sx.region_bytes[which] + (pay_off - sx.region_off[which]) + (size_t)e * 4;
          snd[0] = pay[0]; snd[1] = pay[1]; snd[2] = pay[2]; snd[3] = pay[3];
        }
      }
      if (!sx.pack_only) store_factor<RP>(L, which, row, col, sum / (float)W);
    }
    return;
  } else {
    const int NW = CH * bits / 32;       // 32-bit words of one worker's stream in this chunk
    const int e0 = ch.chunk * CH;
    const int cnt = min(CH, count - e0);
    const bool valid = tid < cnt;
    const int e = e0 + tid;
    const int row = valid ? e / r : 0, col = valid ? e % r : 0;
    if (cs) s = S.scol[col];
    const bool s_ok = (s > 0.f) && (s < INFINITY);
    const size_t nbytes_total = ((size_t)count * bits + 7) / 8;
    const size_t byte0 = (size_t)ch.chunk * (CH / 8) * bits;
    const int nbytes = (int)min((size_t)(CH / 8) * bits, nbytes_total - byte0);
    int Ssum = 0;
    float Sv = 0.f;          // value-domain variant: sum of the workers' dequantised levels, in worker order

    for (int w0 = 0; w0 < W; w0 += WB) {
      const int wn = min(WB, W - w0);
      float x[WB];
#pragma unroll
      for (int u = 0; u < WB; ++u) x[u] = xfirst[u];
      if (w0 + WB < W) {           // the next round's values set out before this round is quantised and packed
#pragma unroll
        for (int u = 0; u < WB; ++u)
          xfirst[u] = (valid && w0 + WB + u < W) ? ld_in<COH>(src + ((size_t)(w0 + WB + u) * rows + row) * RP + col) : 0.f;
      }
      if (tid < CH) {
#pragma unroll
        for (int u = 0; u < WB; ++u) {
          if (u < wn) {
            int k = 0;      // k = #{i : |x| / s >= thr[i]}, thr ascending, NLEV - 1 = 2^(B-1) - 1 entries
            if (s_ok && valid) {
              if constexpr (kRegThr) {
                const float tt = __fdiv_rn(fabsf(x[u]), s);
#pragma unroll
                for (int i = 0; i < kNThr; ++i) k += (tt >= thr_r[i]) ? 1 : 0;
              } else {
                k = level_of_call(x[u], s, S.thr, NLEV);
              }
            }
            const int neg = (valid && x[u] < 0.f) ? 1 : 0;
            S.codes[u][tid] = (uint8_t)((neg << (bits - 1)) | k);   // 0 beyond the factor's end: pads the last byte
            const int sk = neg ? -k : k;
            Ssum += sk;
            if (qt.avg_values) Sv += __ldg(qt.deq + sk + (NLEV - 1));
          }
        }
      }
      __syncthreads();
      // little-endian bit stream: word j of the chunk holds bits [32 j, 32 j + 32) = the codes of
      // elements 32 j / B .. (32 j + 31) / B
      for (int task = tid; task < wn * NW; task += NT) {
        const int u = task / NW, j = task - u * NW;
        const int bit0 = 32 * j;
        const int q0 = bit0 / bits;
        uint32_t word = 0;
        if constexpr (B == 4) {
          // eight codes per word, one per byte in shared memory (each below 16): byte pairs to nibble pairs, twice
          const uint32_t* cw = reinterpret_cast<const uint32_t*>(&S.codes[u][8 * j]);
          auto nib = [](uint32_t x) { x = (x | (x >> 4)) & 0x00FF00FFu; return (x | (x >> 8)) & 0xFFFFu; };
          word = nib(cw[0]) | (nib(cw[1]) << 16);
        } else if constexpr (B == 8) {
          word = *reinterpret_cast<const uint32_t*>(&S.codes[u][4 * j]);
        } else {
#pragma unroll
        for (int i = 0; i < 32 / bits + 2; ++i) {
          const int q = q0 + i;
          const int sh = q * bits - bit0;
          if (sh < 32) {
            const uint32_t c = S.codes[u][min(q, CH + 3)];
            word |= (sh >= 0) ? (c << sh) : (c >> (-sh));
          }
        }
        }
        const int nb = min(4, nbytes - 4 * j);       // bytes of this word inside the stream
        uint8_t* pay = t.payload + (size_t)(w0 + u) * t.payload_stride + pay_off + byte0 + 4 * j;
        uint8_t* snd = sx.pack_only
            ? sx.send[which] + (size_t)(w0 + u) * sx.region_bytes[which] + (pay_off - sx.region_off[which]) + byte0 + 4 * j
            : nullptr;
        if (nb == 4 && (reinterpret_cast<uintptr_t>(pay) & 3) == 0) *reinterpret_cast<uint32_t*>(pay) = word;
        else
          for (int i = 0; i < nb; ++i) pay[i] = (uint8_t)(word >> (8 * i));
        if (snd) {           // the same stream, contiguous over the local workers, for the all-gather
          if (nb == 4 && (reinterpret_cast<uintptr_t>(snd) & 3) == 0) *reinterpret_cast<uint32_t*>(snd) = word;
          else
            for (int i = 0; i < nb; ++i) snd[i] = (uint8_t)(word >> (8 * i));
        }
      }
      __syncthreads();
    }

    if (valid && !sx.pack_only) {
      float v = 0.f;
      if (s_ok) v = qt.avg_values ? s * (Sv / (float)W) : s * __ldg(qt.deq + Ssum + W * (NLEV - 1));
      store_factor<RP>(L, which, row, col, v);
    }
  }
}

// ---------------------------------------------------------------------------------------
// The same exchange for a block of consecutive factor rows, results only: out[lr][j] (shared memory,
// [nrows][RP]) = the dequantised worker average of rows first_row .. first_row + nrows - 1 of P (which = 0) or
// of Q (which = 1).  No codes are packed and nothing is written to global memory: this is for a CTA that needs
// P_bar or Q_bar of its own rows at once (the one-launch round), while the chunk jobs above write payload and
// state off the critical path.  Same arithmetic in the same order, hence the same bits as exchange_body.
// ---------------------------------------------------------------------------------------
template <int RP, int NT> struct ExchangeLocalSmem {
  float thr[128];
  float sred[NT / 32];
  float scol[RP];
};

template <int RP, int NT, bool COH>
__device__ __noinline__ void exchange_rows_local(const Tables& t, const QuantTables& qt, int which, const LayerDev& L,
                                                 int first_row, int nrows, float* out, int tid, void* smem) {
  auto& S = *static_cast<ExchangeLocalSmem<RP, NT>*>(smem);
  const int bits = qt.bits;
  const int NLEV = (bits == 32) ? 2 : 1 << (bits - 1);
  const int W = t.W, r = L.r;
  const int rows = which ? L.m : L.n;
  const int nblk = which ? L.nqb : L.npb;
  const float* __restrict__ maxes = which ? L.maxq : L.maxp;
  const float* __restrict__ src = (which ? L.Qw : L.P) + (size_t)first_row * RP;   // [W][rows][RP], from the block's first row
  const size_t plane = (size_t)rows * RP;
  const int count = nrows * RP;
  for (int i = tid; i < NLEV - 1; i += NT) S.thr[i] = qt.thr[i];
  float s = 0.f;
  const bool cs = t.col_scales != 0;
  if (bits != 32) {
    if (cs) {
      if (tid < RP) S.scol[tid] = 0.f;
      __syncthreads();
      for (int i = tid; i < W * nblk * RP; i += NT) s = fmaxf(s, ld_in<COH>(maxes + i));
      atomicMax(reinterpret_cast<int*>(S.scol) + tid % RP, __float_as_int(s));      // non-negative floats order like their bits
      __syncthreads();
    } else {
      for (int i = tid; i < W * nblk; i += NT) s = fmaxf(s, ld_in<COH>(maxes + i));
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) s = fmaxf(s, __shfl_xor_sync(0xffffffffu, s, o));
      if ((tid & 31) == 0) S.sred[tid >> 5] = s;
      __syncthreads();
      s = S.sred[0];
      for (int i = 1; i < NT / 32; ++i) s = fmaxf(s, S.sred[i]);
    }
  } else {
    __syncthreads();
  }
  // A thread takes its elements EB at a time; the worker loop is rolled (small code: this runs once per launch
  // from a cold instruction cache) with the next worker's EB values already on their way.
  constexpr int EB = 4;
#pragma unroll 1
  for (int e0 = tid; e0 < count; e0 += EB * NT) {
    const float* px[EB];
    float sj[EB], xc[EB], fsum[EB], Sv[EB];
    int Ssum[EB];
    bool on[EB];
#pragma unroll
    for (int i = 0; i < EB; ++i) {
      const int e = e0 + i * NT, j = e % RP;
      on[i] = e < count && j < r;
      px[i] = src + e;
      sj[i] = cs ? S.scol[j] : s;
      if (!((sj[i] > 0.f) && (sj[i] < INFINITY)) && bits != 32) on[i] = false;      // zero or non-finite scale: the average is 0
      xc[i] = on[i] ? ld_in<COH>(px[i]) : 0.f;
      fsum[i] = 0.f; Sv[i] = 0.f; Ssum[i] = 0;
    }
#pragma unroll 1
    for (int w = 0; w < W; ++w) {
      float xn[EB];
#pragma unroll
      for (int i = 0; i < EB; ++i) xn[i] = (on[i] && w + 1 < W) ? ld_in<COH>(px[i] + (size_t)(w + 1) * plane) : 0.f;
#pragma unroll
      for (int i = 0; i < EB; ++i) {
        if (on[i]) {
          if (bits == 32) fsum[i] += xc[i];
          else {
            const int k = level_of_call(xc[i], sj[i], S.thr, NLEV);
            const int sk = (xc[i] < 0.f) ? -k : k;
            Ssum[i] += sk;
            if (qt.avg_values) Sv[i] += __ldg(qt.deq + sk + (NLEV - 1));
          }
        }
        xc[i] = xn[i];
      }
    }
#pragma unroll
    for (int i = 0; i < EB; ++i) {
      const int e = e0 + i * NT;
      if (e < count) {
        float v = 0.f;
        if (on[i]) {
          if (bits == 32) v = fsum[i] / (float)W;
          else v = qt.avg_values ? sj[i] * (Sv[i] / (float)W) : sj[i] * __ldg(qt.deq + Ssum[i] + W * (NLEV - 1));
        }
        out[e] = v;
      }
    }
  }
  __syncthreads();
}

}  // namespace
}  // namespace lqsgd

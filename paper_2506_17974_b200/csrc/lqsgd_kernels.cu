// sm_100a kernels of the LQ-SGD round (Algorithm 1, loop body).
//
// Three streaming passes over the n x m data carry all the HBM traffic:
//   pass 1: M = G + E (Eq. 8) written over E, partial P = M Q          (power step)
//   pass 2: partial Q = M^T P_bar                                        (second power step)
//   pass 3: G_hat = P_bar Q_bar^T (Eq. 6), E = M - G_hat (Eq. 7)
// The products are rank-r updates of a stream.  The kernels of this file do them on CUDA cores
// with fp32 accumulation: a few FMAs per byte up to r = 8 (layers with 16-byte aligned rows then
// run on the bulk-copy staged versions in lqsgd_stream.cu); above that the tensor-core passes of
// lqsgd_tc.cu take the aligned layers and these kernels keep the rest.
// Between the passes small kernels finish the factors: fixed-order reduction of the partial
// sums, CholeskyQR in fp64 (Orthonormalize), scale, LogQuantize (Eq. 4 through a threshold
// table), bit-packing, the exact integer worker sum, LogDequantize (Eq. 5 through a table).
//
// Every kernel is a persistent or table-driven grid: CTAs walk a tile table the host planned
// once, so a 64 x 27 layer costs a table entry, not a launch.  Nothing here spins or waits on
// another CTA, and every reduction has a fixed order: results are bit-reproducible.
#include "lqsgd_dev.h"

#include <cuda_bf16.h>

#include <math.h>

namespace lqsgd {
namespace {

// ---------------------------------------------------------------------------------------
// small helpers
// ---------------------------------------------------------------------------------------
template <int N>
__device__ __forceinline__ void load_contig_ro(const float* __restrict__ p, float (&out)[N]) {
  // N contiguous read-only floats, aligned to min(N,4)*4 bytes, through the read-only path
  if constexpr (N % 4 == 0) {
#pragma unroll
    for (int i = 0; i < N / 4; ++i) {
      float4 v = __ldg(reinterpret_cast<const float4*>(p) + i);
      out[4 * i] = v.x; out[4 * i + 1] = v.y; out[4 * i + 2] = v.z; out[4 * i + 3] = v.w;
    }
  } else if constexpr (N == 2) {
    float2 v = __ldg(reinterpret_cast<const float2*>(p));
    out[0] = v.x; out[1] = v.y;
  } else {
#pragma unroll
    for (int i = 0; i < N; ++i) out[i] = __ldg(p + i);
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

// Packed fp32 arithmetic of sm_100: one instruction, two fused multiply-adds on a register pair,
// d.lo = a.lo * b.lo + c.lo and d.hi likewise, each half rounded exactly like fmaf.  Pass 2 at
// rank 8 issues 8 multiply-adds per 4 bytes it streams and is bound by instruction issue, not by
// HBM, unless they go out in pairs.
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

// VEC consecutive floats of a streamed matrix row (VEC = 4: one 128-bit access, VEC = 1: scalar).
template <int VEC>
struct Pack {
  float v[VEC];
};

template <int VEC>
__device__ __forceinline__ Pack<VEC> ld_stream(const float* p) {   // read once: evict first
  Pack<VEC> r;
  if constexpr (VEC == 4) {
    float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    r.v[0] = t.x; r.v[1] = t.y; r.v[2] = t.z; r.v[3] = t.w;
  } else {
    r.v[0] = __ldcs(p);
  }
  return r;
}

template <int VEC>
__device__ __forceinline__ Pack<VEC> ld_l2(const float* p) {       // keep in L2, skip L1
  Pack<VEC> r;
  if constexpr (VEC == 4) {
    float4 t = __ldcg(reinterpret_cast<const float4*>(p));
    r.v[0] = t.x; r.v[1] = t.y; r.v[2] = t.z; r.v[3] = t.w;
  } else {
    r.v[0] = __ldcg(p);
  }
  return r;
}

// Streamed load that asks L2 to keep the line (the next pass starts on the data this pass reads last).
template <int VEC>
__device__ __forceinline__ Pack<VEC> ld_keep(const float* p, uint64_t pol) {
  Pack<VEC> r;
  if constexpr (VEC == 4) {
    asm("ld.global.cg.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]) : "l"(p), "l"(pol));
  } else {
    asm("ld.global.cg.L2::cache_hint.f32 %0, [%1], %2;" : "=f"(r.v[0]) : "l"(p), "l"(pol));
  }
  return r;
}

template <int VEC>
__device__ __forceinline__ Pack<VEC> ld_ro(const float* __restrict__ p) {   // read-only data, cached in L1
  Pack<VEC> r;
  if constexpr (VEC == 4) {
    float4 t = __ldg(reinterpret_cast<const float4*>(p));
    r.v[0] = t.x; r.v[1] = t.y; r.v[2] = t.z; r.v[3] = t.w;
  } else {
    r.v[0] = __ldg(p);
  }
  return r;
}

// q[k * RP + j] = Q[col + k][j] for k < VEC, read from the transposed copy Qt[j][col + k] so
// that the lanes of a warp (consecutive columns) read consecutive addresses.
template <int RP, int VEC>
__device__ __forceinline__ void load_q_slice(const float* __restrict__ Qt, int mt, int col, float (&q)[VEC * RP]) {
#pragma unroll
  for (int j = 0; j < RP; ++j) {
    const Pack<VEC> v = ld_ro<VEC>(Qt + (size_t)j * mt + col);
#pragma unroll
    for (int k = 0; k < VEC; ++k) q[k * RP + j] = v.v[k];
  }
}

template <int VEC>
__device__ __forceinline__ void st_default(float* p, const Pack<VEC>& x) {
  if constexpr (VEC == 4) *reinterpret_cast<float4*>(p) = make_float4(x.v[0], x.v[1], x.v[2], x.v[3]);
  else *p = x.v[0];
}

template <int VEC>
__device__ __forceinline__ void st_stream(float* p, const Pack<VEC>& x) {
  if constexpr (VEC == 4) __stcs(reinterpret_cast<float4*>(p), make_float4(x.v[0], x.v[1], x.v[2], x.v[3]));
  else __stcs(p, x.v[0]);
}

// Sum of v[i] over the 32 lanes for every i, in log steps that halve the live values:
// afterwards lane l holds the totals of indices [l*N/32, (l+1)*N/32) when N >= 32, and the
// total of index l / (32/N) when N < 32 (in v[0 .. max(N/32,1))).  Fixed order: deterministic.
template <int N, int O>
__device__ __forceinline__ void warp_transpose_reduce(float* v, int lane) {
  if constexpr (O >= 1) {
    if constexpr (N > 1) {
      constexpr int H = N / 2;
      const bool up = (lane & O) != 0;
#pragma unroll
      for (int i = 0; i < H; ++i) {
        const float a = v[i], b = v[i + H];
        const float send = up ? a : b;
        const float keep = up ? b : a;
        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, O);
      }
      warp_transpose_reduce<H, O / 2>(v, lane);
    } else {
      v[0] += __shfl_xor_sync(0xffffffffu, v[0], O);
      warp_transpose_reduce<1, O / 2>(v, lane);
    }
  }
}

// ---------------------------------------------------------------------------------------
// pass 1: M = G + E over E (Eq. 8), partial P = M Q (Alg. 1 power step)
// A tile is up to 32 rows x one column chunk; each warp owns 4 rows, lanes stride the columns,
// every lane accumulates 4 x RP partial dot products and the warp reduces them at the end.
// ---------------------------------------------------------------------------------------
template <int RP, int VEC>
__device__ __forceinline__ void pass1_tile(const Tables& t, const Tile& tl) {
  const LayerDev& L = t.layers[tl.layer];
  const int m = L.m;
  const float* __restrict__ G = t.grads[(size_t)tl.layer * t.W + tl.worker];
  float* __restrict__ E = L.E + (size_t)tl.worker * L.n * m;
  const float* __restrict__ Qt = L.Qt;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r0 = tl.row0 + warp * 4;
  const int nr = min(4, tl.row0 + tl.nrows - r0);   // rows this warp owns (may be <= 0)
  if (nr <= 0) return;
  const int cend = tl.col0 + tl.ncols;
  constexpr int STEP = 32 * VEC;

  float acc[4 * RP];
#pragma unroll
  for (int i = 0; i < 4 * RP; ++i) acc[i] = 0.f;

  Pack<VEC> g[4], e[4];
  int c = tl.col0 + lane * VEC;
  auto fetch = [&](int col, Pack<VEC>(&gg)[4], Pack<VEC>(&ee)[4]) {
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      if (a < nr) {
        const size_t off = (size_t)(r0 + a) * m + col;
        gg[a] = ld_stream<VEC>(G + off);
        ee[a] = ld_stream<VEC>(E + off);
      }
    }
  };
  if (c < cend) fetch(c, g, e);
  for (; c < cend; c += STEP) {
    Pack<VEC> gn[4], en[4];
    const int cn = c + STEP;
    if (cn < cend) fetch(cn, gn, en);       // next column group in flight before this one is stored
    float q[VEC * RP];
    load_q_slice<RP, VEC>(Qt, L.mt, c, q);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      if (a < nr) {
        Pack<VEC> mv;
#pragma unroll
        for (int k = 0; k < VEC; ++k) mv.v[k] = g[a].v[k] + e[a].v[k];
        st_default<VEC>(E + (size_t)(r0 + a) * m + c, mv);
#pragma unroll
        for (int k = 0; k < VEC; ++k)
#pragma unroll
          for (int j = 0; j < RP; ++j) acc[a * RP + j] = fmaf(mv.v[k], q[k * RP + j], acc[a * RP + j]);
      }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) { g[a] = gn[a]; e[a] = en[a]; }
  }

  constexpr int N = 4 * RP;
  warp_transpose_reduce<N, 16>(acc, lane);
  float* Pp = L.Ppart + ((size_t)tl.worker * L.ncc + tl.part) * (size_t)L.n * RP;
  if constexpr (N >= 32) {
    constexpr int PER = N / 32;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int idx = lane * PER + i;
      const int a = idx / RP, j = idx % RP;
      if (a < nr) Pp[(size_t)(r0 + a) * RP + j] = acc[i];
    }
  } else {
    constexpr int DUP = 32 / N;
    const int idx = lane / DUP;
    const int a = idx / RP, j = idx % RP;
    if ((lane % DUP) == 0 && a < nr) Pp[(size_t)(r0 + a) * RP + j] = acc[0];
  }
}

template <int RP>
__global__ void __launch_bounds__(kPassThreads, (RP <= 8 ? 2 : 1))
pass1_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles) {
  pdl_wait();
  clear_status_words(t);
  for (int i = blockIdx.x; i < ntiles; i += gridDim.x) {
    const Tile tl = tiles[i];
    if constexpr (RP > 16) pass1_tile<RP, 1>(t, tl);   // above rank 16 these kernels only take what the tensor-core passes cannot
    else if (t.layers[tl.layer].vec) pass1_tile<RP, 4>(t, tl);
    else pass1_tile<RP, 1>(t, tl);
  }
}

// ---------------------------------------------------------------------------------------
// Column-owner mapping shared by pass 2 and pass 3: a tile is nrows x up to 128*VEC columns.
// Thread = (row group g, vector column cv); groups interleave the tile's rows.
// ---------------------------------------------------------------------------------------
struct ColMap {
  int cwv, cw, ng, g, cv;
  bool active;
};

template <int VEC>
__device__ __forceinline__ ColMap col_map(const Tile& tl) {
  ColMap cm;
  cm.cwv = (tl.ncols + VEC - 1) / VEC;       // vector columns in the tile (<= 128)
  cm.cw = (cm.cwv + 31) & ~31;                // rounded to whole warps
  cm.ng = kPassThreads / cm.cw;               // row groups
  cm.g = threadIdx.x / cm.cw;
  cm.cv = threadIdx.x % cm.cw;
  cm.active = cm.g < cm.ng && cm.cv < cm.cwv;
  return cm;
}

// ---------------------------------------------------------------------------------------
// pass 2: partial Q = M^T P_bar (Alg. 1, second product).  Each thread owns VEC columns and
// accumulates VEC x RP sums over its group's rows; P_bar rows are warp-uniform loads.
// Row groups are then summed through shared memory in group order.
// ---------------------------------------------------------------------------------------
template <int RP, int VEC>
__device__ __forceinline__ void pass2_tile(const Tables& t, const Tile& tl, float* red, float* pb, uint64_t pol) {
  const LayerDev& L = t.layers[tl.layer];
  const int m = L.m;
  const float* __restrict__ M = L.E + (size_t)tl.worker * L.n * m;
  const float* __restrict__ Pbar = L.Pbar;
  const ColMap cm = col_map<VEC>(tl);
  const int col = tl.col0 + cm.cv * VEC;
  const int rend = tl.row0 + tl.nrows;

  float acc[VEC * RP];
#pragma unroll
  for (int i = 0; i < VEC * RP; ++i) acc[i] = 0.f;

  constexpr bool kPaired = RP >= 2 && RP <= 8 && VEC == 4;
  if constexpr (kPaired) {
    // the tile's rows of P_bar wait in shared memory: every thread needs every row, and reading them
    // there leaves the L1 path to the stream of M (158 instead of 191 us on 8192 x 25088 at rank 8)
    constexpr int VW = RP < 4 ? RP : 4;
    for (int e = threadIdx.x; e < tl.nrows * (RP / VW); e += kPassThreads) {
      float v[VW];
      load_contig_ro<VW>(Pbar + (size_t)tl.row0 * RP + (size_t)e * VW, v);
      store_contig<VW>(pb + (size_t)e * VW, v);
    }
    __syncthreads();
  }
  if (cm.active) {
    constexpr int U = 8;
    int i = tl.row0 + cm.g;
    if constexpr (kPaired) {
      // the sums of columns j, j + 1 of P_bar travel as a pair: half the multiply-add instructions
      constexpr int H = RP / 2;
      uint64_t acc2[VEC * H];
#pragma unroll
      for (int k = 0; k < VEC * H; ++k) acc2[k] = 0ull;                      // (+0, +0)
      auto row_update = [&](const Pack<VEC>& mv, int row) {
        float p[RP];
        if constexpr (RP >= 4) {
#pragma unroll
          for (int q4 = 0; q4 < RP / 4; ++q4) {
            const float4 v = reinterpret_cast<const float4*>(pb + (size_t)(row - tl.row0) * RP)[q4];
            p[4 * q4] = v.x; p[4 * q4 + 1] = v.y; p[4 * q4 + 2] = v.z; p[4 * q4 + 3] = v.w;
          }
        } else {
          const float2 v = *reinterpret_cast<const float2*>(pb + (size_t)(row - tl.row0) * RP);
          p[0] = v.x; p[1] = v.y;
        }
        uint64_t p2[H];
#pragma unroll
        for (int jj = 0; jj < H; ++jj) p2[jj] = pack2(p[2 * jj], p[2 * jj + 1]);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
          const uint64_t mk = pack2(mv.v[k], mv.v[k]);
#pragma unroll
          for (int jj = 0; jj < H; ++jj) acc2[k * H + jj] = fma2(mk, p2[jj], acc2[k * H + jj]);
        }
      };
      for (; i + (U - 1) * cm.ng < rend; i += U * cm.ng) {
        Pack<VEC> mv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) mv[u] = ld_keep<VEC>(M + (size_t)(i + u * cm.ng) * m + col, pol);
#pragma unroll
        for (int u = 0; u < U; ++u) row_update(mv[u], i + u * cm.ng);
      }
      for (; i < rend; i += cm.ng) row_update(ld_keep<VEC>(M + (size_t)i * m + col, pol), i);
#pragma unroll
      for (int k = 0; k < VEC; ++k)
#pragma unroll
        for (int jj = 0; jj < H; ++jj) unpack2(acc2[k * H + jj], acc[k * RP + 2 * jj], acc[k * RP + 2 * jj + 1]);
    } else {
    for (; i + (U - 1) * cm.ng < rend; i += U * cm.ng) {
      Pack<VEC> mv[U];
#pragma unroll
      for (int u = 0; u < U; ++u) mv[u] = ld_keep<VEC>(M + (size_t)(i + u * cm.ng) * m + col, pol);
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float p[RP];
        load_contig_ro<RP>(Pbar + (size_t)(i + u * cm.ng) * RP, p);
#pragma unroll
        for (int k = 0; k < VEC; ++k)
#pragma unroll
          for (int j = 0; j < RP; ++j) acc[k * RP + j] = fmaf(mv[u].v[k], p[j], acc[k * RP + j]);
      }
    }
    for (; i < rend; i += cm.ng) {
      const Pack<VEC> mv = ld_keep<VEC>(M + (size_t)i * m + col, pol);
      float p[RP];
      load_contig_ro<RP>(Pbar + (size_t)i * RP, p);
#pragma unroll
      for (int k = 0; k < VEC; ++k)
#pragma unroll
        for (int j = 0; j < RP; ++j) acc[k * RP + j] = fmaf(mv.v[k], p[j], acc[k * RP + j]);
    }
    }
  }
  // fixed-order sum over the row groups: group gg hands its sums to group 0
  for (int gg = 1; gg < cm.ng; ++gg) {
    __syncthreads();
    if (cm.active && cm.g == gg) {
#pragma unroll
      for (int k = 0; k < VEC * RP; ++k) red[k * cm.cw + cm.cv] = acc[k];
    }
    __syncthreads();
    if (cm.active && cm.g == 0) {
#pragma unroll
      for (int k = 0; k < VEC * RP; ++k) acc[k] += red[k * cm.cw + cm.cv];
    }
  }
  if (cm.active && cm.g == 0) {
    float* dst = L.Qpart + (((size_t)tl.worker * L.nrb + tl.part) * (size_t)m + col) * RP;
    store_contig<VEC * RP>(dst, acc);
  }
  __syncthreads();   // red is reused by the next tile
}

template <int RP>
__global__ void __launch_bounds__(kPassThreads, (RP <= 2 ? 4 : (RP <= 8 ? 3 : 1)))
pass2_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles) {
  pdl_wait();
  __shared__ float red[128 * (RP > 16 ? 1 : 4) * RP];
  __shared__ __align__(16) float pb[(RP >= 2 && RP <= 8) ? (RP <= 4 ? 128 : 32 * RP) * RP : 4];   // a tile's rows of P_bar: up to max(128, 32 RP)
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  for (int i = blockIdx.x; i < ntiles; i += gridDim.x) {
    const Tile tl = tiles[i];
    if constexpr (RP > 16) pass2_tile<RP, 1>(t, tl, red, pb, pol);
    else if (t.layers[tl.layer].vec) pass2_tile<RP, 4>(t, tl, red, pb, pol);
    else pass2_tile<RP, 1>(t, tl, red, pb, pol);
  }
}

// ---------------------------------------------------------------------------------------
// pass 3: G_hat = P_bar Q_bar^T (Eq. 6) once per layer, E_w = M_w - G_hat (Eq. 7) per worker.
// Each thread keeps its VEC rows of Q_bar in registers, forms G_hat for 4 rows at a time and
// walks the workers with the next worker's M already in flight.
// ---------------------------------------------------------------------------------------
template <int RP, int VEC>
__device__ __forceinline__ void pass3_tile(const Tables& t, const Tile& tl) {
  const LayerDev& L = t.layers[tl.layer];
  const int m = L.m, W = t.W;
  const size_t plane = (size_t)L.n * m;
  float* __restrict__ E = L.E;
  float* __restrict__ Gh = t.ghat[tl.layer];                                  // may be null
  float* __restrict__ Wt = t.weights ? t.weights[tl.layer] : nullptr;         // may be null
  const float lr = t.lr;
  const float* __restrict__ Pbar = L.Pbar;
  const ColMap cm = col_map<VEC>(tl);
  if (!cm.active) return;
  const int col = tl.col0 + cm.cv * VEC;
  const int rend = tl.row0 + tl.nrows;

  float q[VEC * RP];
  load_q_slice<RP, VEC>(L.Qt, L.mt, col, q);

  constexpr int RB = 4;
  const int rstep = RB * cm.ng;
  auto fetch = [&](int i0, int w, Pack<VEC>(&mv)[RB]) {
#pragma unroll
    for (int u = 0; u < RB; ++u) {
      const int i = i0 + u * cm.ng;
      if (i < rend) mv[u] = ld_stream<VEC>(E + (size_t)w * plane + (size_t)i * m + col);
    }
  };
  int i0 = tl.row0 + cm.g;
  Pack<VEC> cur[RB];
  if (i0 < rend) fetch(i0, 0, cur);
  for (; i0 < rend; i0 += rstep) {
    Pack<VEC> gh[RB];
#pragma unroll
    for (int u = 0; u < RB; ++u) {
      const int i = i0 + u * cm.ng;
      if (i < rend) {
        float p[RP];
        load_contig_ro<RP>(Pbar + (size_t)i * RP, p);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
          float s = 0.f;
#pragma unroll
          for (int j = 0; j < RP; ++j) s = fmaf(p[j], q[k * RP + j], s);
          gh[u].v[k] = s;
        }
        if (Gh) st_stream<VEC>(Gh + (size_t)i * m + col, gh[u]);
        if (Wt) {                                  // model update of Alg. 1: w <- w - lr * G_hat
          Pack<VEC> wv = ld_stream<VEC>(Wt + (size_t)i * m + col);
#pragma unroll
          for (int k = 0; k < VEC; ++k) wv.v[k] = fmaf(-lr, gh[u].v[k], wv.v[k]);
          st_stream<VEC>(Wt + (size_t)i * m + col, wv);
        }
      }
    }
    for (int w = 0; w < W; ++w) {
      Pack<VEC> nxt[RB];
      if (w + 1 < W) fetch(i0, w + 1, nxt);
      else if (i0 + rstep < rend) fetch(i0 + rstep, 0, nxt);
#pragma unroll
      for (int u = 0; u < RB; ++u) {
        const int i = i0 + u * cm.ng;
        if (i < rend) {
          Pack<VEC> ev;
#pragma unroll
          for (int k = 0; k < VEC; ++k) ev.v[k] = cur[u].v[k] - gh[u].v[k];
          st_stream<VEC>(E + (size_t)w * plane + (size_t)i * m + col, ev);
        }
      }
#pragma unroll
      for (int u = 0; u < RB; ++u) cur[u] = nxt[u];
    }
  }
}

template <int RP>
__global__ void __launch_bounds__(kPassThreads, (RP <= 8 ? 2 : 1))
pass3_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles) {
  pdl_wait();
  for (int i = blockIdx.x; i < ntiles; i += gridDim.x) {
    const Tile tl = tiles[i];
    if constexpr (RP > 16) pass3_tile<RP, 1>(t, tl);
    else if (t.layers[tl.layer].vec) pass3_tile<RP, 4>(t, tl);
    else pass3_tile<RP, 1>(t, tl);
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

template <int RP>
__global__ void __launch_bounds__(256)
p_reduce_gram_kernel(Tables t, const FactorBlock* __restrict__ fbs) {
  pdl_wait();
  __shared__ double rows[kFactorBlockRows][RP];     // the block's rows, converted once
  const FactorBlock fb = fbs[blockIdx.x];
  const LayerDev& L = t.layers[fb.layer];
  const int n = L.n;
  const int tid = threadIdx.x;
  if (tid < kFactorBlockRows) {
    const int row = fb.blk * kFactorBlockRows + tid;
    float p[RP];
#pragma unroll
    for (int j = 0; j < RP; ++j) p[j] = 0.f;
    if (row < n) {
      const float* src = L.Ppart + ((size_t)fb.worker * L.ncc * n + row) * RP;
      // the partials' loads go out together (8 at a time); the additions keep the chunk order
      int cc = 0;
      if constexpr (RP <= 8) {
        for (; cc + 8 <= L.ncc; cc += 8) {
          float v[8][RP];
#pragma unroll
          for (int u = 0; u < 8; ++u) load_contig_ro<RP>(src + (size_t)(cc + u) * n * RP, v[u]);
#pragma unroll
          for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int j = 0; j < RP; ++j) p[j] += v[u][j];
        }
      }
      for (; cc < L.ncc; ++cc) {
        float v[RP];
        load_contig_ro<RP>(src + (size_t)cc * n * RP, v);
#pragma unroll
        for (int j = 0; j < RP; ++j) p[j] += v[j];
      }
      if (L.ncc > 1) store_contig<RP>(L.Praw + ((size_t)fb.worker * n + row) * RP, p);
    }
#pragma unroll
    for (int j = 0; j < RP; ++j) rows[tid][j] = (double)p[j];
  }
  __syncthreads();
  for (int e = tid; e < RP * RP; e += 256) {
    const int i = e / RP, j = e % RP;
    if (j < i) continue;                                 // the Gram matrix is symmetric: upper triangle, mirrored
    double s = 0.0;
    for (int k = 0; k < kFactorBlockRows; ++k) s = fma(rows[k][i], rows[k][j], s);
    double* gp = L.gram_part + ((size_t)fb.worker * L.npb + fb.blk) * (RP * RP);
    gp[i * RP + j] = s;
    gp[j * RP + i] = s;
  }
}

// Gram = sum of the block Grams (block order), Cholesky  Gram = L L^T  (R = L^T), by a whole CTA;
// every CTA that orthonormalises a block of rows redoes this small factorisation itself, which
// costs less than a kernel boundary.  Lf (shared, RP*RP doubles, row-major) receives L, invd the
// reciprocals of its diagonal, dead[j] = 1 for a column dropped as dependent (its row and column
// of L are then those of the identity).  Returns true if any column was dropped.
template <int RP>
__device__ __forceinline__ bool cholesky_factor(double (*A)[RP + 1], int r, double* Lf, double* invd, int* dead);

template <int RP>
__device__ __forceinline__ bool cholesky_lower(const LayerDev& L, int worker, double* Lf, double* invd, int* dead) {
  __shared__ double A[RP][RP + 1];     // Gram, overwritten by L (lower triangle)
  const int tid = threadIdx.x, nt = blockDim.x;
  // Gram = sum of the block Grams.  With more threads than entries the blocks are dealt to SEG
  // segments (segment g takes blocks g, g + SEG, ...), eight loads in flight each; the segments'
  // sums are then added in segment order: a fixed order, and a chain SEG times shorter.
  constexpr int SEG = (RP * RP <= 64) ? 128 / (RP * RP) : 1;      // the factor kernels run 128 threads
  if constexpr (SEG > 1) {
    __shared__ double segsum[SEG][RP * RP];
    if (tid < SEG * RP * RP) {
      const int e = tid % (RP * RP), g = tid / (RP * RP);
      const double* gp = L.gram_part + (size_t)worker * L.npb * (RP * RP) + e;
      double s = 0.0;
      int b = g;
      for (; b + 7 * SEG < L.npb; b += 8 * SEG) {
        double x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = gp[(size_t)(b + u * SEG) * (RP * RP)];
#pragma unroll
        for (int u = 0; u < 8; ++u) s += x[u];
      }
      for (; b < L.npb; b += SEG) s += gp[(size_t)b * (RP * RP)];
      segsum[g][e] = s;
    }
    __syncthreads();
    if (tid < RP * RP) {
      double s = segsum[0][tid];
#pragma unroll
      for (int g = 1; g < SEG; ++g) s += segsum[g][tid];
      A[tid / RP][tid % RP] = s;
    }
  } else {
    for (int e = tid; e < RP * RP; e += nt) {
      const double* gp = L.gram_part + (size_t)worker * L.npb * (RP * RP) + e;
      double s = 0.0;
      int b = 0;
      for (; b + 8 <= L.npb; b += 8) {        // eight loads in flight, additions in block order
        double x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = gp[(size_t)(b + u) * (RP * RP)];
#pragma unroll
        for (int u = 0; u < 8; ++u) s += x[u];
      }
      for (; b < L.npb; ++b) s += gp[(size_t)b * (RP * RP)];
      A[e / RP][e % RP] = s;
    }
  }
  __syncthreads();
  return cholesky_factor<RP>(A, L.r, Lf, invd, dead);
}

// Cholesky of the Gram matrix in A (shared, complete and visible to the CTA on entry).
template <int RP>
__device__ __forceinline__ bool cholesky_factor(double (*A)[RP + 1], int r, double* Lf, double* invd, int* dead) {
  __shared__ double diag0[RP];
  const int tid = threadIdx.x, nt = blockDim.x;
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
  for (int e = tid; e < RP * RP; e += nt) {
    const int i = e / RP, k = e % RP;
    Lf[e] = (k <= i && i < r) ? A[i][k] : 0.0;
  }
  int any = 0;
  for (int j = 0; j < r; ++j) any |= dead[j];
  __syncthreads();
  return any != 0;
}

__device__ __forceinline__ float block_max_128(float v, float* sm) {
  // max over a 128-thread block; NaN compares false and is dropped (reported separately)
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
  __syncthreads();
  return fmaxf(fmaxf(sm[0], sm[1]), fmaxf(sm[2], sm[3]));
}

template <int RP>
__global__ void __launch_bounds__(kFactorBlockRows)
p_apply_kernel(Tables t, const FactorBlock* __restrict__ fbs) {
  pdl_wait();
  __shared__ double Lf[RP * RP];
  __shared__ double invd[RP];
  __shared__ int dead[RP];
  __shared__ float smax[4];
  __shared__ float scol[4][RP];
  const FactorBlock fb = fbs[blockIdx.x];
  const LayerDev& L = t.layers[fb.layer];
  const int n = L.n, tid = threadIdx.x;
  const bool dropped = cholesky_lower<RP>(L, fb.worker, Lf, invd, dead);
  if (dropped && fb.blk == 0 && tid == 0) atomicOr(&t.status[fb.layer], 1u);
  const int row = fb.blk * kFactorBlockRows + tid;
  float amax = 0.f;
  float o[RP];
#pragma unroll
  for (int j = 0; j < RP; ++j) o[j] = 0.f;
  if (row < n) {
    // the row of P solves  o R = p  with R = L^T upper triangular: forward substitution in fp64,
    //   o[j] = (p[j] - sum_{k<j} o[k] L[j][k]) / L[j][j];   a dropped column gives 0
    float p[RP];
    load_contig_ro<RP>(L.Praw + ((size_t)fb.worker * n + row) * RP, p);
    double od[RP];
    bool bad = false;
#pragma unroll
    for (int j = 0; j < RP; ++j) {
      double s = (double)p[j];
#pragma unroll
      for (int k = 0; k < j; ++k) s = fma(-od[k], Lf[j * RP + k], s);
      od[j] = (j < L.r && !dead[j]) ? s * invd[j] : 0.0;
      o[j] = (float)od[j];
      amax = fmaxf(amax, fabsf(o[j]));
      bad |= !(fabsf(o[j]) < INFINITY);
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
      if ((tid & 31) == 0) scol[tid >> 5][j] = v;
    }
    __syncthreads();
    if (tid < RP)
      L.maxp[((size_t)fb.worker * L.npb + fb.blk) * RP + tid] =
          fmaxf(fmaxf(scol[0][tid], scol[1][tid]), fmaxf(scol[2][tid], scol[3][tid]));
    return;
  }
  amax = block_max_128(amax, smax);
  if (tid == 0) L.maxp[(size_t)fb.worker * L.npb + fb.blk] = amax;
}

// Orthonormalize for a layer of at most 512 rows (every layer of the ResNet-18 set), one CTA per
// (layer, worker), one thread per row: the sum of pass 1's column-chunk partials, the Gram matrix in
// fp64 (every entry summed over eight 64-row segments, the segments then added in order), its
// Cholesky factor, the rows of P by substitution and the block maxima: what p_reduce_gram and
// p_apply do in two launches for taller layers.
constexpr int kOrthSmallRows = 512;
template <int RP>
__global__ void __launch_bounds__(kOrthSmallRows, 3)   // three CTAs per SM: 444 at once, one wave for 21 layers x 16 workers
p_orth_small_kernel(Tables t, const FactorBlock* __restrict__ fbs) {
  pdl_wait();
  constexpr int NE = RP * RP, NSEG = 8, SEGROWS = kOrthSmallRows / NSEG;
  __shared__ double rows[kOrthSmallRows][RP];
  __shared__ double seg[NSEG][NE];
  __shared__ double A[RP][RP + 1];
  __shared__ double Lf[NE];
  __shared__ double invd[RP];
  __shared__ int dead[RP];
  __shared__ float wmax[kOrthSmallRows / 32][RP];
  const FactorBlock fb = fbs[blockIdx.x];
  const LayerDev& L = t.layers[fb.layer];
  const int n = L.n, tid = threadIdx.x, row = tid;
  float p[RP];
#pragma unroll
  for (int j = 0; j < RP; ++j) p[j] = 0.f;
  if (row < n) {
    const float* src = L.Ppart + ((size_t)fb.worker * L.ncc * n + row) * RP;
    for (int cc = 0; cc < L.ncc; ++cc) {
      float v[RP];
      load_contig_ro<RP>(src + (size_t)cc * n * RP, v);
#pragma unroll
      for (int j = 0; j < RP; ++j) p[j] += v[j];
    }
    if (L.ncc > 1) store_contig<RP>(L.Praw + ((size_t)fb.worker * n + row) * RP, p);
  }
#pragma unroll
  for (int j = 0; j < RP; ++j) rows[tid][j] = (double)p[j];
  __syncthreads();
  for (int idx = tid; idx < NSEG * NE; idx += kOrthSmallRows) {
    const int e = idx % NE, g = idx / NE, i = e / RP, j = e % RP;
    if (j < i) continue;                                   // upper triangle; mirrored below
    double s = 0.0;
    for (int k = g * SEGROWS; k < (g + 1) * SEGROWS; ++k) s = fma(rows[k][i], rows[k][j], s);
    seg[g][e] = s;
  }
  __syncthreads();
  if (tid < NE) {
    const int i = tid / RP, j = tid % RP;
    if (j >= i) {
      double s = seg[0][tid];
#pragma unroll
      for (int g = 1; g < NSEG; ++g) s += seg[g][tid];
      A[i][j] = s;
      A[j][i] = s;
    }
  }
  __syncthreads();
  const bool dropped = cholesky_factor<RP>(A, L.r, Lf, invd, dead);
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
      for (int k = 0; k < j; ++k) s = fma(-od[k], Lf[j * RP + k], s);
      od[j] = (j < L.r && !dead[j]) ? s * invd[j] : 0.0;
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
    if ((tid & 31) == 0) wmax[tid >> 5][j] = v;
  }
  __syncthreads();
  const int ncs = t.col_scales ? RP : 1;
  if (tid < L.npb * ncs) {
    const int blk = tid / ncs, j0 = tid % ncs;
    float a = 0.f;
    for (int w4 = 4 * blk; w4 < 4 * blk + 4; ++w4)
      for (int j = (t.col_scales ? j0 : 0); j < (t.col_scales ? j0 + 1 : RP); ++j) a = fmaxf(a, wmax[w4][j]);
    L.maxp[((size_t)fb.worker * L.npb + blk) * ncs + j0] = a;
  }
}

// Q_w = sum of the row-chunk partials of pass 2, in chunk order; block max |Q_w|.  A thread owns
// V = min(RP, 4) consecutive columns of a row (one 128-bit load per partial when RP >= 4) and the
// loads of several partials are in flight together: the chain of nrb dependent additions, not a
// chain of nrb memory latencies, is what a row costs.
template <int RP> struct QReduceThreads { static constexpr int value = RP >= 8 ? 256 : 128; };   // one item per thread up to rank 8
template <int RP>
__global__ void __launch_bounds__(QReduceThreads<RP>::value)
q_reduce_kernel(Tables t, const FactorBlock* __restrict__ fbs) {
  pdl_wait();
  constexpr int kQReduceThreads = QReduceThreads<RP>::value;
  constexpr int V = RP < 4 ? RP : 4;        // floats per thread item
  constexpr int TPR = RP / V;               // items per row: 1, 2, 4 or 8 (divides the block size and 32)
  __shared__ float smax[kQReduceThreads / 32][TPR * V];
  const FactorBlock fb = fbs[blockIdx.x];
  const LayerDev& L = t.layers[fb.layer];
  const int m = L.m, tid = threadIdx.x, nrb = L.nrb;
  const size_t plane = (size_t)m * RP;      // floats of one partial
  float cmax[V];
#pragma unroll
  for (int v = 0; v < V; ++v) cmax[v] = 0.f;
  bool bad = false;
  for (int item = tid; item < kFactorBlockRows * TPR; item += kQReduceThreads) {
    const int row = fb.blk * kFactorBlockRows + item / TPR;
    if (row >= m) break;
    const size_t off = (size_t)row * RP + (size_t)(item % TPR) * V;
    const float* src = L.Qpart + (size_t)fb.worker * nrb * plane + off;
    float q[V];
#pragma unroll
    for (int v = 0; v < V; ++v) q[v] = 0.f;
    int rb = 0;
    for (; rb + 8 <= nrb; rb += 8) {
      float x[8][V];
#pragma unroll
      for (int u = 0; u < 8; ++u) load_contig_ro<V>(src + (size_t)(rb + u) * plane, x[u]);
#pragma unroll
      for (int u = 0; u < 8; ++u)
#pragma unroll
        for (int v = 0; v < V; ++v) q[v] += x[u][v];
    }
    for (; rb < nrb; ++rb) {
      float x[V];
      load_contig_ro<V>(src + (size_t)rb * plane, x);
#pragma unroll
      for (int v = 0; v < V; ++v) q[v] += x[v];
    }
    if (nrb > 1) store_contig<V>(L.Qw + (size_t)fb.worker * plane + off, q);
#pragma unroll
    for (int v = 0; v < V; ++v) {
      cmax[v] = fmaxf(cmax[v], fabsf(q[v]));
      bad |= !(fabsf(q[v]) < INFINITY);
    }
  }
  if (bad) atomicOr(&t.status[fb.layer], 8u);
  // maxima: the columns a thread owns are fixed (256 and 32 are multiples of TPR): columns (tid % TPR) V + v
  const int warp = tid >> 5, lane = tid & 31;
  if (t.col_scales) {
#pragma unroll
    for (int v = 0; v < V; ++v) {
#pragma unroll
      for (int o = 16; o >= TPR; o >>= 1) cmax[v] = fmaxf(cmax[v], __shfl_xor_sync(0xffffffffu, cmax[v], o));
      if (lane < TPR) smax[warp][lane * V + v] = cmax[v];
    }
    __syncthreads();
    if (tid < RP) {
      float a = smax[0][tid];
#pragma unroll
      for (int w = 1; w < kQReduceThreads / 32; ++w) a = fmaxf(a, smax[w][tid]);
      L.maxq[((size_t)fb.worker * L.nqb + fb.blk) * RP + tid] = a;
    }
    return;
  }
  float amax = cmax[0];
#pragma unroll
  for (int v = 1; v < V; ++v) amax = fmaxf(amax, cmax[v]);
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if (lane == 0) smax[warp][0] = amax;
  __syncthreads();
  if (tid == 0) {
#pragma unroll
    for (int w = 1; w < kQReduceThreads / 32; ++w) amax = fmaxf(amax, smax[w][0]);
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
// each worker's payload.  One block = 256 entries of one tensor.  Runs as a kernel of its own or
// as extra blocks of the exchange of P (same block shape), which saves a launch per round.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void vectors_block(const VectorJob& vj, int blk, uint8_t* payload, uint64_t payload_stride,
                                              int W) {
  const ExchangeChunk ch = vj.chunks[blk];
  const VectorDev v = vj.vecs[ch.layer];
  const int i = ch.chunk * 256 + threadIdx.x;
  if (i >= v.len) return;
  float s = 0.f;
  for (int w = 0; w < W; ++w) {
    const float x = vj.vgrads[(size_t)ch.layer * W + w][i];
    reinterpret_cast<float*>(payload + (size_t)w * payload_stride + v.pay_off)[i] = x;
    s += x;
  }
  const float mean = s / (float)vj.W_total;     // with workers on other GPUs too: this rank's share of the mean
  if (vj.vghat[ch.layer]) vj.vghat[ch.layer][i] = mean;
  if (vj.vweights && vj.vweights[ch.layer]) vj.vweights[ch.layer][i] = fmaf(-vj.lr, mean, vj.vweights[ch.layer][i]);
}
__global__ void __launch_bounds__(256)
vectors_kernel(VectorJob vj, uint8_t* payload, uint64_t payload_stride, int W) {
  pdl_wait();
  vectors_block(vj, blockIdx.x, payload, payload_stride, W);
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
// ---------------------------------------------------------------------------------------
// B = bits per code (2..8), or 32: quantiser bypassed.  One block = 256 factor elements.
template <int RP, int B>
__global__ void __launch_bounds__(256)
exchange_kernel(Tables t, QuantTables qt, int which, const ExchangeChunk* __restrict__ chunks, int nchunks,
                SplitExchange sx, VectorJob vj) {
  pdl_wait();
  if ((int)blockIdx.x >= nchunks) {      // blocks past the factor chunks: the round's 1-D tensors
    vectors_block(vj, (int)blockIdx.x - nchunks, t.payload, t.payload_stride, t.W);
    return;
  }
  constexpr int CH = kExchangeChunk;   // 256 factor elements per block, one per thread
  constexpr int WB = 8;                // workers handled per round
  constexpr int NLEV = (B == 32) ? 2 : 1 << (B - 1);
  __shared__ float thr[128];
  __shared__ __align__(4) uint8_t codes[WB][CH + 4];
  __shared__ float sred[8];
  __shared__ float scol8[8][RP];
  __shared__ float scol[RP];
  const ExchangeChunk ch = chunks[blockIdx.x];
  const LayerDev& L = t.layers[ch.layer];
  const int W = t.W, tid = threadIdx.x;
  const int rows = which ? L.m : L.n, r = L.r;
  const int count = rows * r;
  const int nblk = which ? L.nqb : L.npb;
  const float* __restrict__ maxes = which ? L.maxq : L.maxp;
  const float* __restrict__ src = which ? L.Qw : L.P;   // [W][rows][RP]
  const uint64_t pay_off = which ? L.pay_q_off : L.pay_p_off;

  for (int i = tid; i < NLEV - 1; i += 256) thr[i] = qt.thr[i];
  if (tid < WB) *reinterpret_cast<uint32_t*>(&codes[tid][CH]) = 0u;     // what a word task reads past the chunk
  float s = 0.f;
  const bool cs = t.col_scales != 0;
  if (cs) {
    // variant: one scale per column.  Block maxima are [W][nblk][RP]; thread tid only meets column tid % RP.
    for (int i = tid; i < W * nblk * RP; i += 256) s = fmaxf(s, __ldg(maxes + i));
#pragma unroll
    for (int o = 16; o >= RP; o >>= 1) s = fmaxf(s, __shfl_xor_sync(0xffffffffu, s, o));
    if ((tid & 31) < RP) scol8[tid >> 5][tid & 31] = s;
    __syncthreads();
    if (tid < RP) {
      float a = scol8[0][tid];
#pragma unroll
      for (int i = 1; i < 8; ++i) a = fmaxf(a, scol8[i][tid]);
      scol[tid] = a;
    }
    __syncthreads();
  } else {
    for (int i = tid; i < W * nblk; i += 256) s = fmaxf(s, __ldg(maxes + i));
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) s = fmaxf(s, __shfl_xor_sync(0xffffffffu, s, o));
    if ((tid & 31) == 0) sred[tid >> 5] = s;
    __syncthreads();
    s = sred[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) s = fmaxf(s, sred[i]);
    if (sx.pack_only) s = sx.scales[which * sx.n_mat + ch.layer];   // scale agreed between the ranks
  }
  // scales, status: once per layer
  if (ch.chunk == 0 && (cs ? tid < r : tid == 0)) {
    const float sj = cs ? scol[tid] : s;
    L.scales[cs ? which * RP + tid : which] = sj;
    for (int w = 0; w < W; ++w) {
      float* ps = reinterpret_cast<float*>(t.payload + (size_t)w * t.payload_stride + L.pay_scale_off);
      ps[cs ? which * r + tid : which] = sj;
    }
    if (B != 32 && !(sj > 0.f)) atomicOr(&t.status[ch.layer], which ? 4u : 2u);
    if (!(sj < INFINITY)) atomicOr(&t.status[ch.layer], 8u);
  }

  if constexpr (B == 32) {
    // Quantiser bypassed (plain PowerSGD exchange): the factor travels as fp32 and the workers'
    // factors are averaged directly (Eq. 1), in worker order.
    const int e = ch.chunk * CH + tid;
    if (e < count) {
      const int row = e / r, col = e - row * r;
      float sum = 0.f;
      for (int w = 0; w < W; ++w) {
        const float x = __ldg(src + ((size_t)w * rows + row) * RP + col);
        sum += x;
        uint8_t* pay = t.payload + (size_t)w * t.payload_stride + pay_off + (size_t)e * 4;
        const unsigned bits32 = __float_as_uint(x);               // the stream may start on any byte
        pay[0] = bits32 & 0xff; pay[1] = (bits32 >> 8) & 0xff; pay[2] = (bits32 >> 16) & 0xff; pay[3] = bits32 >> 24;
      }
      store_factor<RP>(L, which, row, col, sum / (float)W);
    }
    return;
  } else {
    constexpr int NW = CH * B / 32;      // 32-bit words of one worker's stream in this chunk
    const int e0 = ch.chunk * CH;
    const int cnt = min(CH, count - e0);
    const bool valid = tid < cnt;
    const int e = e0 + tid;
    const int row = valid ? e / r : 0, col = valid ? e % r : 0;
    if (cs) s = scol[col];
    const bool s_ok = (s > 0.f) && (s < INFINITY);
    const size_t nbytes_total = ((size_t)count * B + 7) / 8;
    const size_t byte0 = (size_t)ch.chunk * (CH / 8) * B;
    const int nbytes = (int)min((size_t)(CH / 8) * B, nbytes_total - byte0);
    int S = 0;
    float Sv = 0.f;          // value-domain variant: sum of the workers' dequantised levels, in worker order

    for (int w0 = 0; w0 < W; w0 += WB) {
      const int wn = min(WB, W - w0);
      float x[WB];
#pragma unroll
      for (int u = 0; u < WB; ++u)
        x[u] = (valid && u < wn) ? __ldg(src + ((size_t)(w0 + u) * rows + row) * RP + col) : 0.f;
#pragma unroll
      for (int u = 0; u < WB; ++u) {
        if (u < wn) {
          int k = 0;
          if (s_ok && valid) {
            const float tt = __fdiv_rn(fabsf(x[u]), s);
            // k = #{i : tt >= thr[i]}, thr ascending, NLEV - 1 = 2^(B-1) - 1 entries: B - 1 halving steps
#pragma unroll
            for (int step = NLEV / 2; step >= 1; step >>= 1)
              if (tt >= thr[k + step - 1]) k += step;
          }
          const int neg = (valid && x[u] < 0.f) ? 1 : 0;
          codes[u][tid] = (uint8_t)((neg << (B - 1)) | k);   // 0 beyond the factor's end: pads the last byte
          const int sk = neg ? -k : k;
          S += sk;
          if (qt.avg_values) Sv += __ldg(qt.deq + sk + (NLEV - 1));
        }
      }
      __syncthreads();
      // little-endian bit stream: word j of the chunk holds bits [32 j, 32 j + 32) = the codes of
      // elements 32 j / B .. (32 j + 31) / B
      for (int task = tid; task < wn * NW; task += 256) {
        const int u = task / NW, j = task - u * NW;
        const int bit0 = 32 * j;
        const int q0 = bit0 / B;
        uint32_t word = 0;
#pragma unroll
        for (int i = 0; i < 32 / B + 2; ++i) {
          const int q = q0 + i;
          const int sh = q * B - bit0;
          if (sh < 32) {
            const uint32_t c = codes[u][min(q, CH + 3)];
            word |= (sh >= 0) ? (c << sh) : (c >> (-sh));
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
      if (s_ok) v = qt.avg_values ? s * (Sv / (float)W) : s * __ldg(qt.deq + S + W * (NLEV - 1));
      store_factor<RP>(L, which, row, col, v);
    }
  }
}

// One worker's unpacked codes (one per byte) from its packed stream: what lqsgd_get_state returns
// for LQSGD_STATE_CODES_*.
__global__ void __launch_bounds__(256)
unpack_codes_kernel(const uint8_t* __restrict__ stream, int count, int b, uint8_t* __restrict__ out) {
  const int e = blockIdx.x * 256 + threadIdx.x;
  if (e >= count) return;
  const size_t nbytes = ((size_t)count * b + 7) / 8;
  const size_t bit = (size_t)e * b, byte = bit >> 3;
  const int sh = (int)(bit & 7);
  unsigned v = stream[byte];
  if (sh + b > 8 && byte + 1 < nbytes) v |= (unsigned)stream[byte + 1] << 8;
  out[e] = (uint8_t)((v >> sh) & ((1u << b) - 1u));
}

// Qt[j][i] = Q[i][j]: refreshes the transposed copy after Q was set from outside.
__global__ void __launch_bounds__(256)
q_transpose_kernel(const float* __restrict__ Q, float* __restrict__ Qt, float* __restrict__ Qcat, int m, int RP, int mt,
                   int kcat, int tc) {
  pdl_wait();
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= m) return;
  for (int j = 0; j < RP; ++j) {
    const float v = Q[(size_t)i * RP + j];
    Qt[(size_t)j * mt + i] = v;
    if (tc) {
      const float lo = tf32_remainder(v);
      Qt[(size_t)(RP + j) * mt + i] = lo;
      float* qc = Qcat + (size_t)i * kcat + j;
      qc[0] = v; qc[RP] = lo; qc[2 * RP] = v;
    }
  }
}

// ---------------------------------------------------------------------------------------
// Split exchange, for workers spread over several GPUs (the All-Reduce of Alg. 1 as a real
// exchange): every rank reduces its block maxima to one local scale per layer
// (scale_reduce_kernel), the ranks agree on the maximum, each packs its workers' codes with that
// scale (exchange_kernel in pack-only mode), the packed streams are all-gathered, and
// sum_dequant_kernel adds the signed levels of ALL workers (exact integers) and applies Eq. 5.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
scale_reduce_kernel(Tables t, int which, float* scales, int n_mat) {
  pdl_wait();
  __shared__ float sred[8];
  const int layer = blockIdx.x, tid = threadIdx.x;
  const LayerDev& L = t.layers[layer];
  const int nblk = which ? L.nqb : L.npb;
  const float* __restrict__ maxes = which ? L.maxq : L.maxp;
  float s = 0.f;
  for (int i = tid; i < t.W * nblk; i += 256) s = fmaxf(s, maxes[i]);
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) s = fmaxf(s, __shfl_xor_sync(0xffffffffu, s, o));
  if ((tid & 31) == 0) sred[tid >> 5] = s;
  __syncthreads();
  if (tid == 0) {
    for (int i = 1; i < 8; ++i) s = fmaxf(s, sred[i]);
    scales[which * n_mat + layer] = fmaxf(s, sred[0]);
  }
}

template <int RP>
__global__ void __launch_bounds__(256)
sum_dequant_kernel(Tables t, QuantTables qt, int which, const ExchangeChunk* __restrict__ chunks, SplitExchange sx,
                   const uint8_t* __restrict__ gathered, int n_streams) {
  pdl_wait();
  const ExchangeChunk ch = chunks[blockIdx.x];
  const LayerDev& L = t.layers[ch.layer];
  const int tid = threadIdx.x, b = qt.bits;
  const int nlev = 1 << (b - 1);
  const int rows = which ? L.m : L.n, r = L.r;
  const int count = rows * r;
  const int e = ch.chunk * kExchangeChunk + tid;
  const float s = sx.scales[which * sx.n_mat + ch.layer];
  const bool s_ok = (s > 0.f) && (s < INFINITY);
  if (e < count) {
    const uint64_t off = (which ? L.pay_q_off : L.pay_p_off) - sx.region_off[which];   // this layer's stream
    const size_t nbytes = ((size_t)count * b + 7) / 8;
    const size_t bit = (size_t)e * b, byte = bit >> 3;
    const int sh = (int)(bit & 7);
    int S = 0;
    float Sv = 0.f;
    for (int w = 0; w < n_streams; ++w) {
      const uint8_t* st = gathered + (size_t)w * sx.region_bytes[which] + off;
      unsigned v = st[byte];
      if (sh + b > 8 && byte + 1 < nbytes) v |= (unsigned)st[byte + 1] << 8;
      const unsigned code = (v >> sh) & ((1u << b) - 1u);
      const int k = (int)(code & (unsigned)(nlev - 1));
      const int sk = (code >> (b - 1)) ? -k : k;
      S += sk;
      if (qt.avg_values) Sv += __ldg(qt.deq + sk + (nlev - 1));
    }
    float v = 0.f;
    if (s_ok) v = qt.avg_values ? s * (Sv / (float)n_streams) : s * __ldg(qt.deq + S + n_streams * (nlev - 1));
    const int row = e / r, col = e - row * r;
    store_factor<RP>(L, which, row, col, v);
  }
  if (ch.chunk == 0 && tid == 0) {
    L.scales[which] = s;
    for (int w = 0; w < t.W; ++w) {
      float* ps = reinterpret_cast<float*>(t.payload + (size_t)w * t.payload_stride + L.pay_scale_off);
      ps[which] = s;
    }
    if (!(s > 0.f)) atomicOr(&t.status[ch.layer], which ? 4u : 2u);
    if (!(s < INFINITY)) atomicOr(&t.status[ch.layer], 8u);
  }
}

// Variant (LQSGD_FLAG_QUANTIZE_VECTORS): a 1-D tensor goes through the factor exchange, one CTA per
// tensor: scale = max over workers and entries, code = sign | level (Eq. 4), little-endian b-bit
// stream per worker, exact integer sum of the signed levels (or, value-domain variant, the sum of the
// dequantised levels), Eq. 5 once.  Entries are taken 256 at a time, 8 workers per round.
template <int B>
__global__ void __launch_bounds__(256)
vectors_quant_kernel(const VectorDev* __restrict__ vecs, const float* const* __restrict__ vgrads,
                     float* const* __restrict__ vghat, float* const* __restrict__ vweights, float lr, uint8_t* payload,
                     uint64_t payload_stride, int W, QuantTables qt) {
  pdl_wait();
  constexpr int CH = 256, WB = 8, NLEV = 1 << (B - 1), NW = CH * B / 32;
  __shared__ float thr[128];
  __shared__ __align__(4) uint8_t codes[WB][CH + 4];
  __shared__ float sred[8];
  const VectorDev v = vecs[blockIdx.x];
  const int tid = threadIdx.x, len = v.len;
  for (int i = tid; i < NLEV - 1; i += 256) thr[i] = qt.thr[i];
  if (tid < WB) *reinterpret_cast<uint32_t*>(&codes[tid][CH]) = 0u;
  float s = 0.f;
  for (int w = 0; w < W; ++w) {
    const float* g = vgrads[(size_t)blockIdx.x * W + w];
    for (int i = tid; i < len; i += 256) s = fmaxf(s, fabsf(g[i]));
  }
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) s = fmaxf(s, __shfl_xor_sync(0xffffffffu, s, o));
  if ((tid & 31) == 0) sred[tid >> 5] = s;
  __syncthreads();
  s = sred[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) s = fmaxf(s, sred[i]);
  const bool s_ok = (s > 0.f) && (s < INFINITY);
  if (tid == 0)
    for (int w = 0; w < W; ++w) *reinterpret_cast<float*>(payload + (size_t)w * payload_stride + v.pay_scale_off) = s;
  const size_t nbytes_total = ((size_t)len * B + 7) / 8;
  float* gh = vghat[blockIdx.x];
  float* wt = vweights ? vweights[blockIdx.x] : nullptr;
  for (int e0 = 0; e0 < len; e0 += CH) {
    const bool valid = e0 + tid < len;
    const size_t byte0 = (size_t)(e0 / 8) * B;
    const int nbytes = (int)min((size_t)(CH / 8) * B, nbytes_total - byte0);
    int S = 0;
    float Sv = 0.f;
    for (int w0 = 0; w0 < W; w0 += WB) {
      const int wn = min(WB, W - w0);
#pragma unroll
      for (int u = 0; u < WB; ++u) {
        if (u < wn) {
          const float x = valid ? vgrads[(size_t)blockIdx.x * W + w0 + u][e0 + tid] : 0.f;
          int k = 0;
          if (s_ok && valid) {
            const float tt = __fdiv_rn(fabsf(x), s);
#pragma unroll
            for (int step = NLEV / 2; step >= 1; step >>= 1)
              if (tt >= thr[k + step - 1]) k += step;
          }
          const int neg = (valid && x < 0.f) ? 1 : 0;
          codes[u][tid] = (uint8_t)((neg << (B - 1)) | k);
          const int sk = neg ? -k : k;
          S += sk;
          if (qt.avg_values) Sv += __ldg(qt.deq + sk + (NLEV - 1));
        }
      }
      __syncthreads();
      for (int task = tid; task < wn * NW; task += 256) {
        const int u = task / NW, j = task - u * NW;
        const int bit0 = 32 * j, q0 = bit0 / B;
        uint32_t word = 0;
#pragma unroll
        for (int i = 0; i < 32 / B + 2; ++i) {
          const int q = q0 + i, sh = q * B - bit0;
          if (sh < 32) {
            const uint32_t c = codes[u][min(q, CH + 3)];
            word |= (sh >= 0) ? (c << sh) : (c >> (-sh));
          }
        }
        const int nb = min(4, nbytes - 4 * j);
        uint8_t* pay = payload + (size_t)(w0 + u) * payload_stride + v.pay_off + byte0 + 4 * j;
        for (int i = 0; i < nb; ++i) pay[i] = (uint8_t)(word >> (8 * i));
      }
      __syncthreads();
    }
    if (valid) {
      float mean = 0.f;
      if (s_ok) mean = qt.avg_values ? s * (Sv / (float)W) : s * __ldg(qt.deq + S + W * (NLEV - 1));
      if (gh) gh[e0 + tid] = mean;
      if (wt) wt[e0 + tid] = fmaf(-lr, mean, wt[e0 + tid]);
    }
  }
}

}  // namespace

// ---------------------------------------------------------------------------------------
// host launchers: dispatch on the padded rank RP in {1, 2, 4, 8, 16, 32}
// ---------------------------------------------------------------------------------------
#define LQSGD_DISPATCH_RP(RPV, ...)                 \
  switch (RPV) {                                    \
    case 1: { constexpr int RP = 1; __VA_ARGS__; } break;   \
    case 2: { constexpr int RP = 2; __VA_ARGS__; } break;   \
    case 4: { constexpr int RP = 4; __VA_ARGS__; } break;   \
    case 8: { constexpr int RP = 8; __VA_ARGS__; } break;   \
    case 16: { constexpr int RP = 16; __VA_ARGS__; } break; \
    case 32: { constexpr int RP = 32; __VA_ARGS__; } break; \
    default: return cudaErrorInvalidValue;          \
  }

cudaError_t launch_pass1(int rp, const Tables& t, const Tile* tiles, int ntiles, Launch l) {
  if (ntiles == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP(rp, (launch_pdl(pass1_kernel<RP>, l.grid, kPassThreads, 0, l.stream, t, tiles, ntiles)));
  return cudaGetLastError();
}

cudaError_t launch_q_transpose(const float* Q, float* Qt, float* Qcat, int m, int RP, int mt, int kcat, int tc,
                               cudaStream_t stream) {
  launch_pdl(q_transpose_kernel, (m + 255) / 256, 256, 0, stream, Q, Qt, Qcat, m, RP, mt, kcat, tc);
  return cudaGetLastError();
}

cudaError_t launch_pass2(int rp, const Tables& t, const Tile* tiles, int ntiles, Launch l) {
  if (ntiles == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP(rp, (launch_pdl(pass2_kernel<RP>, l.grid, kPassThreads, 0, l.stream, t, tiles, ntiles)));
  return cudaGetLastError();
}

cudaError_t launch_pass3(int rp, const Tables& t, const Tile* tiles, int ntiles, Launch l) {
  if (ntiles == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP(rp, (launch_pdl(pass3_kernel<RP>, l.grid, kPassThreads, 0, l.stream, t, tiles, ntiles)));
  return cudaGetLastError();
}

cudaError_t launch_p_reduce_gram(int rp, const Tables& t, const FactorBlock* fb, int nfb, Launch l) {
  if (nfb == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP(rp, (launch_pdl(p_reduce_gram_kernel<RP>, nfb, 256, 0, l.stream, t, fb)));
  return cudaGetLastError();
}

cudaError_t launch_p_apply(int rp, const Tables& t, const FactorBlock* fb, int nfb, Launch l) {
  if (nfb == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP(rp, (launch_pdl(p_apply_kernel<RP>, nfb, kFactorBlockRows, 0, l.stream, t, fb)));
  return cudaGetLastError();
}

cudaError_t launch_p_orth_small(int rp, const Tables& t, const FactorBlock* fb, int nfb, Launch l) {
  if (nfb == 0) return cudaSuccess;
  switch (rp) {
    case 1: launch_pdl(p_orth_small_kernel<1>, nfb, kOrthSmallRows, 0, l.stream, t, fb); break;
    case 2: launch_pdl(p_orth_small_kernel<2>, nfb, kOrthSmallRows, 0, l.stream, t, fb); break;
    case 4: launch_pdl(p_orth_small_kernel<4>, nfb, kOrthSmallRows, 0, l.stream, t, fb); break;
    case 8: launch_pdl(p_orth_small_kernel<8>, nfb, kOrthSmallRows, 0, l.stream, t, fb); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_q_reduce(int rp, const Tables& t, const FactorBlock* fb, int nfb, Launch l) {
  if (nfb == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP(rp, (launch_pdl(q_reduce_kernel<RP>, nfb, QReduceThreads<RP>::value, 0, l.stream, t, fb)));
  return cudaGetLastError();
}

cudaError_t launch_exchange(int rp, int which, const Tables& t, const QuantTables& q,
                            const ExchangeChunk* ch, int nch, const SplitExchange& sx, const VectorJob* ride, Launch l) {
  if (nch == 0) return cudaSuccess;
  const VectorJob vj = ride ? *ride : VectorJob{};
  const int grid = nch + vj.nchunks;
#define LQSGD_EXCHANGE_BITS(BV) case BV: launch_pdl(exchange_kernel<RP, BV>, grid, 256, 0, l.stream, t, q, which, ch, nch, sx, vj); break;
  LQSGD_DISPATCH_RP(rp, {
    switch (q.bits) {
      LQSGD_EXCHANGE_BITS(2) LQSGD_EXCHANGE_BITS(3) LQSGD_EXCHANGE_BITS(4) LQSGD_EXCHANGE_BITS(5)
      LQSGD_EXCHANGE_BITS(6) LQSGD_EXCHANGE_BITS(7) LQSGD_EXCHANGE_BITS(8) LQSGD_EXCHANGE_BITS(32)
      default: return cudaErrorInvalidValue;
    }
  });
#undef LQSGD_EXCHANGE_BITS
  return cudaGetLastError();
}

cudaError_t launch_unpack_codes(const uint8_t* stream, int count, int bits, uint8_t* out, cudaStream_t st) {
  if (count == 0) return cudaSuccess;
  unpack_codes_kernel<<<(count + 255) / 256, 256, 0, st>>>(stream, count, bits, out);
  return cudaGetLastError();
}

cudaError_t launch_scale_reduce(const Tables& t, int which, float* scales, int n_mat, Launch l) {
  if (n_mat == 0) return cudaSuccess;
  launch_pdl(scale_reduce_kernel, n_mat, 256, 0, l.stream, t, which, scales, n_mat);
  return cudaGetLastError();
}

cudaError_t launch_sum_dequant(int rp, int which, const Tables& t, const QuantTables& q, const ExchangeChunk* ch,
                               int nch, const SplitExchange& sx, const uint8_t* gathered, int n_streams, Launch l) {
  if (nch == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP(rp, (launch_pdl(sum_dequant_kernel<RP>, nch, 256, 0, l.stream, t, q, which, ch, sx, gathered,
                                    n_streams)));
  return cudaGetLastError();
}

cudaError_t launch_vectors(const VectorJob& vj, uint8_t* payload, uint64_t payload_stride, int W, Launch l) {
  if (vj.nchunks == 0) return cudaSuccess;
  launch_pdl(vectors_kernel, vj.nchunks, 256, 0, l.stream, vj, payload, payload_stride, W);
  return cudaGetLastError();
}

cudaError_t launch_vectors_quant(const VectorDev* vecs, int nvecs, const float* const* vgrads, float* const* vghat,
                                 float* const* vweights, float lr, uint8_t* payload, uint64_t payload_stride, int W,
                                 const QuantTables& q, Launch l) {
  if (nvecs == 0) return cudaSuccess;
#define LQSGD_VQ_BITS(BV) case BV: launch_pdl(vectors_quant_kernel<BV>, nvecs, 256, 0, l.stream, vecs, vgrads, vghat, vweights, lr, payload, payload_stride, W, q); break;
  switch (q.bits) {
    LQSGD_VQ_BITS(2) LQSGD_VQ_BITS(3) LQSGD_VQ_BITS(4) LQSGD_VQ_BITS(5) LQSGD_VQ_BITS(6) LQSGD_VQ_BITS(7) LQSGD_VQ_BITS(8)
    default: return cudaErrorInvalidValue;
  }
#undef LQSGD_VQ_BITS
  return cudaGetLastError();
}

cudaError_t pass_occupancy(int rp, int* occ1, int* occ2, int* occ3) {
  cudaError_t e = cudaSuccess;
  LQSGD_DISPATCH_RP(rp, {
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(occ1, pass1_kernel<RP>, kPassThreads, 0);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(occ2, pass2_kernel<RP>, kPassThreads, 0);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(occ3, pass3_kernel<RP>, kPassThreads, 0);
  });
  return e;
}

}  // namespace lqsgd

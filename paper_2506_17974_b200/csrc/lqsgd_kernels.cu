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
#include "lqsgd_factor.cuh"

#include <cuda_bf16.h>

#include <math.h>

namespace lqsgd {
namespace {

// ---------------------------------------------------------------------------------------
// small helpers
// ---------------------------------------------------------------------------------------
template <int N>
__device__ __forceinline__ void load_contig_nc(const float* __restrict__ p, float (&out)[N]) { load_contig<N, false>(p, out); }

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
      load_contig_nc<VW>(Pbar + (size_t)tl.row0 * RP + (size_t)e * VW, v);
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
        load_contig_nc<RP>(Pbar + (size_t)(i + u * cm.ng) * RP, p);
#pragma unroll
        for (int k = 0; k < VEC; ++k)
#pragma unroll
          for (int j = 0; j < RP; ++j) acc[k * RP + j] = fmaf(mv[u].v[k], p[j], acc[k * RP + j]);
      }
    }
    for (; i < rend; i += cm.ng) {
      const Pack<VEC> mv = ld_keep<VEC>(M + (size_t)i * m + col, pol);
      float p[RP];
      load_contig_nc<RP>(Pbar + (size_t)i * RP, p);
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
  prefetch_first_tile(t, tiles, ntiles);
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
        load_contig_nc<RP>(Pbar + (size_t)i * RP, p);
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
// The small steps between the passes: one CTA per table entry, bodies in lqsgd_factor.cuh
// (Orthonormalize as CholeskyQR, the factor exchange, the Q_w reduction, the 1-D tensors).
// ---------------------------------------------------------------------------------------
// The work tables (factor blocks, exchange chunks, the layer entries) are written at create and never change: a small
// kernel fetches its entry and its layer's entry into shared memory BEFORE it waits for the kernel in front of it, so
// that these two dependent memory latencies pass under that kernel's tail instead of heading the step's own chain.
__device__ __forceinline__ const LayerDev* stage_layer(const Tables& t, int layer, LayerDev* sL) {
  static_assert(sizeof(LayerDev) % 4 == 0, "copied word by word");
  const uint32_t* src = reinterpret_cast<const uint32_t*>(t.layers + layer);
  uint32_t* dst = reinterpret_cast<uint32_t*>(sL);
  for (int i = threadIdx.x; i < (int)(sizeof(LayerDev) / 4); i += blockDim.x) dst[i] = __ldg(src + i);
  __syncthreads();
  return sL;
}

template <int RP>
__global__ void __launch_bounds__(256)
p_reduce_gram_kernel(Tables t, const FactorBlock* __restrict__ fbs) {
  __shared__ LayerDev sL;
  const FactorBlock fb = fbs[blockIdx.x];
  const LayerDev* L = stage_layer(t, fb.layer, &sL);
  pdl_wait();
  __shared__ __align__(16) unsigned char smem[sizeof(ReduceGramSmem<RP>)];
  p_reduce_gram_body<RP, 256, false>(t, fb, threadIdx.x, smem, L);
}

template <int RP>
__global__ void __launch_bounds__(kFactorBlockRows)
p_apply_kernel(Tables t, const FactorBlock* __restrict__ fbs) {
  __shared__ LayerDev sL;
  const FactorBlock fb = fbs[blockIdx.x];
  const LayerDev* L = stage_layer(t, fb.layer, &sL);
  pdl_wait();
  __shared__ __align__(16) unsigned char smem[sizeof(ApplySmem<RP, kFactorBlockRows>)];
  p_apply_body<RP, kFactorBlockRows, false>(t, fb, threadIdx.x, smem, L);
}

template <int RP>
__global__ void __launch_bounds__(256)
p_chol_kernel(Tables t, const FactorBlock* __restrict__ fbs) {
  __shared__ LayerDev sL;
  const FactorBlock fb = fbs[blockIdx.x];
  const LayerDev* L = stage_layer(t, fb.layer, &sL);
  pdl_wait();
  __shared__ __align__(16) unsigned char smem[sizeof(CholOnceSmem<RP, 256>)];
  p_chol_body<RP, 256, false>(t, fb, threadIdx.x, smem, L);
}

// Many partial sums per layer (a very tall or very wide layer): the sums of groups of kFoldGroup consecutive
// planes, one CTA per group and kFoldElems elements.  Plane order inside a group, eight loads in flight.
template <typename T>
__device__ __forceinline__ void fold_planes(const FoldJob& j, int tid) {
  const T* __restrict__ src = static_cast<const T*>(j.src);
  T* __restrict__ dst = static_cast<T*>(j.dst);
  const size_t plane = j.plane;
  for (uint32_t e = j.e0 + tid; e < j.e0 + kFoldElems && e < j.plane; e += 256) {
    T s = T(0);
    int u0 = 0;
    for (; u0 + 8 <= j.count; u0 += 8) {
      T x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) x[u] = __ldg(src + (size_t)(u0 + u) * plane + e);
#pragma unroll
      for (int u = 0; u < 8; ++u) s += x[u];
    }
    for (; u0 < j.count; ++u0) s += __ldg(src + (size_t)u0 * plane + e);
    dst[e] = s;
  }
}

__global__ void __launch_bounds__(256)
fold_kernel(const FoldJob* __restrict__ jobs) {
  pdl_wait();
  const FoldJob j = jobs[blockIdx.x];
  if (j.is_double) fold_planes<double>(j, threadIdx.x);
  else fold_planes<float>(j, threadIdx.x);
}

template <int RP>
__global__ void __launch_bounds__(kOrthSmallRows, 3)   // three CTAs per SM: 444 at once, one wave for 21 layers x 16 workers
p_orth_small_kernel(Tables t, const FactorBlock* __restrict__ fbs) {
  __shared__ LayerDev sL;
  const FactorBlock fb = fbs[blockIdx.x];
  const LayerDev* L = stage_layer(t, fb.layer, &sL);
  pdl_wait();
  __shared__ __align__(16) unsigned char smem[sizeof(OrthSmallSmem<RP>)];
  p_orth_small_body<RP, false>(t, fb, threadIdx.x, smem, L);
}

template <int RP> struct QReduceThreads { static constexpr int value = RP >= 8 ? 256 : 128; };   // one item per thread up to rank 8
template <int RP>
__global__ void __launch_bounds__(QReduceThreads<RP>::value)
q_reduce_kernel(Tables t, const FactorBlock* __restrict__ fbs) {
  __shared__ LayerDev sL;
  const FactorBlock fb = fbs[blockIdx.x];
  const LayerDev* L = stage_layer(t, fb.layer, &sL);
  pdl_wait();
  constexpr int NT = QReduceThreads<RP>::value;
  __shared__ __align__(16) unsigned char smem[sizeof(QReduceSmem<RP, NT>)];
  q_reduce_body<RP, NT, false>(t, fb, threadIdx.x, smem, L);
}

__global__ void __launch_bounds__(256)
vectors_kernel(VectorJob vj, uint8_t* payload, uint64_t payload_stride, int W) {
  pdl_wait();
  vectors_block(vj, blockIdx.x, threadIdx.x, payload, payload_stride, W);
}

// Factor exchange, one block per chunk of 256 factor elements; blocks past the factor chunks take the
// round's 1-D tensors (same block shape), which saves a launch per round.
template <int RP, int B, bool PLAIN>
__global__ void __launch_bounds__(256)
exchange_kernel(Tables t, QuantTables qt, int which, const ExchangeChunk* __restrict__ chunks, int nchunks,
                SplitExchange sx, VectorJob vj) {
  if ((int)blockIdx.x >= nchunks) {
    pdl_wait();
    vectors_block(vj, (int)blockIdx.x - nchunks, threadIdx.x, t.payload, t.payload_stride, t.W);
    return;
  }
  __shared__ LayerDev sL;
  const ExchangeChunk ch = chunks[blockIdx.x];
  const LayerDev* L = stage_layer(t, ch.layer, &sL);
  pdl_wait();
  __shared__ __align__(16) unsigned char smem[sizeof(ExchangeSmem<RP, 256>)];
  exchange_body<RP, B, 256, false, PLAIN>(t, qt, which, ch, sx, threadIdx.x, smem, L);
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

// Guard blocks between the pieces of the workspace: one block of 64 threads per guard, one word per thread.
__global__ void __launch_bounds__(64)
guards_kernel(char* base, const uint64_t* __restrict__ offs, uint32_t pattern, unsigned long long* result) {
  const uint64_t off = offs[blockIdx.x] + 4ull * threadIdx.x;
  uint32_t* w = reinterpret_cast<uint32_t*>(base + off);
  if (!result) { *w = pattern; return; }
  if (*w != pattern) {
    atomicAdd(result, 1ull);
    atomicMin(result + 1, (unsigned long long)off);
  }
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
template <int RP>
__global__ void __launch_bounds__(256)
scale_reduce_kernel(Tables t, int which, float* scales, int n_mat) {
  pdl_wait();
  __shared__ float sred[8];
  __shared__ float scol[RP];
  const int layer = blockIdx.x, tid = threadIdx.x;
  const LayerDev& L = t.layers[layer];
  const int nblk = which ? L.nqb : L.npb;
  const float* __restrict__ maxes = which ? L.maxq : L.maxp;
  float s = 0.f;
  if (t.col_scales) {              // one scale per column: maxes are [W][nblk][RP]; 256 is a multiple of RP
    if (tid < RP) scol[tid] = 0.f;
    __syncthreads();
    for (int i = tid; i < t.W * nblk * RP; i += 256) s = fmaxf(s, maxes[i]);
    atomicMax(reinterpret_cast<int*>(scol) + tid % RP, __float_as_int(s));     // non-negative floats order like their bits
    __syncthreads();
    if (tid < RP) scales[(size_t)(which * n_mat + layer) * RP + tid] = scol[tid];
    return;
  }
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

// The sum over ALL workers' streams (n_streams of them, rank after rank) and Eq. 5, for one chunk of 256 factor
// elements.  bits = 32: the streams are the fp32 factors themselves, averaged in stream order (Eq. 1).
template <int RP>
__global__ void __launch_bounds__(256)
sum_dequant_kernel(Tables t, QuantTables qt, int which, const ExchangeChunk* __restrict__ chunks, SplitExchange sx,
                   const uint8_t* __restrict__ gathered, int n_streams) {
  pdl_wait();
  const ExchangeChunk ch = chunks[blockIdx.x];
  const LayerDev& L = t.layers[ch.layer];
  const int tid = threadIdx.x, b = qt.bits;
  const int nlev = b == 32 ? 2 : 1 << (b - 1);
  const int rows = which ? L.m : L.n, r = L.r;
  const int count = rows * r;
  const int e = ch.chunk * kExchangeChunk + tid;
  const float* sc = sx.scales + (size_t)(which * sx.n_mat + ch.layer) * sx.ns;
  if (e < count) {
    const int row = e / r, col = e - row * r;
    const uint64_t off = (which ? L.pay_q_off : L.pay_p_off) - sx.region_off[which];   // this layer's stream
    float v = 0.f;
    if (b == 32) {
      float sum = 0.f;
      for (int w = 0; w < n_streams; ++w) {
        const uint8_t* st = gathered + (size_t)w * sx.region_bytes[which] + off + (size_t)e * 4;
        sum += __uint_as_float((unsigned)st[0] | ((unsigned)st[1] << 8) | ((unsigned)st[2] << 16) | ((unsigned)st[3] << 24));
      }
      v = sum / (float)n_streams;
    } else {
      const float s = sc[sx.ns > 1 ? col : 0];
      const bool s_ok = (s > 0.f) && (s < INFINITY);
      const size_t nbytes = ((size_t)count * b + 7) / 8;
      const size_t bit = (size_t)e * b, byte = bit >> 3;
      const int sh = (int)(bit & 7);
      int S = 0;
      float Sv = 0.f;
      for (int w = 0; w < n_streams; ++w) {
        const uint8_t* st = gathered + (size_t)w * sx.region_bytes[which] + off;
        unsigned u = st[byte];
        if (sh + b > 8 && byte + 1 < nbytes) u |= (unsigned)st[byte + 1] << 8;
        const unsigned code = (u >> sh) & ((1u << b) - 1u);
        const int k = (int)(code & (unsigned)(nlev - 1));
        const int sk = (code >> (b - 1)) ? -k : k;
        S += sk;
        if (qt.avg_values) Sv += __ldg(qt.deq + sk + (nlev - 1));
      }
      if (s_ok) v = qt.avg_values ? s * (Sv / (float)n_streams) : s * __ldg(qt.deq + S + n_streams * (nlev - 1));
    }
    store_factor<RP>(L, which, row, col, v);
  }
  if (ch.chunk == 0 && tid < (sx.ns > 1 ? r : 1)) {
    const float s = sc[tid];
    L.scales[sx.ns > 1 ? which * RP + tid : which] = s;
    for (int w = 0; w < t.W; ++w) {
      float* ps = reinterpret_cast<float*>(t.payload + (size_t)w * t.payload_stride + L.pay_scale_off);
      ps[sx.ns > 1 ? which * r + tid : which] = s;
    }
    if (b != 32 && !(s > 0.f)) atomicOr(&t.status[ch.layer], which ? 4u : 2u);
    if (!(s < INFINITY)) atomicOr(&t.status[ch.layer], 8u);
  }
}

// Workers on several GPUs: after the ranks' shares of the 1-D tensors' means have been summed (one all-reduce
// of the flat buffer), the means go to their tensors and into the weights.  One block = 256 entries of one tensor.
__global__ void __launch_bounds__(256)
vectors_finish_kernel(VectorJob vj) {
  pdl_wait();
  const ExchangeChunk ch = vj.chunks[blockIdx.x];
  const VectorDev v = vj.vecs[ch.layer];
  const int i = ch.chunk * 256 + threadIdx.x;
  if (i >= v.len) return;
  const float mean = vj.xvec[(v.pay_off - vj.xvec_base) / 4 + i];
  if (vj.vghat[ch.layer]) vj.vghat[ch.layer][i] = mean;
  if (vj.vweights && vj.vweights[ch.layer]) vj.vweights[ch.layer][i] = fmaf(-vj.lr, mean, vj.vweights[ch.layer][i]);
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
// host launchers: dispatch on the padded rank RP in {1, 2, 4, 8, 16, 32, 64}
// ---------------------------------------------------------------------------------------
#define LQSGD_DISPATCH_RP(RPV, ...)                 \
  switch (RPV) {                                    \
    case 1: { constexpr int RP = 1; __VA_ARGS__; } break;   \
    case 2: { constexpr int RP = 2; __VA_ARGS__; } break;   \
    case 4: { constexpr int RP = 4; __VA_ARGS__; } break;   \
    case 8: { constexpr int RP = 8; __VA_ARGS__; } break;   \
    case 16: { constexpr int RP = 16; __VA_ARGS__; } break; \
    case 32: { constexpr int RP = 32; __VA_ARGS__; } break; \
    case 64: { constexpr int RP = 64; __VA_ARGS__; } break; \
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

cudaError_t launch_p_chol(int rp, const Tables& t, const FactorBlock* fb, int nfb, Launch l) {
  if (nfb == 0) return cudaSuccess;
  switch (rp) {
    case 32: launch_pdl(p_chol_kernel<32>, nfb, 256, 0, l.stream, t, fb); break;
    case 64: launch_pdl(p_chol_kernel<64>, nfb, 256, 0, l.stream, t, fb); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_fold(const FoldJob* jobs, int njobs, Launch l) {
  if (njobs == 0) return cudaSuccess;
  launch_pdl(fold_kernel, njobs, 256, 0, l.stream, jobs);
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
  const bool plain = !t.col_scales && !q.avg_values && !sx.pack_only;
#define LQSGD_EXCHANGE_BITS(BV) case BV: \
    if (plain) launch_pdl(exchange_kernel<RP, BV, true>, grid, 256, 0, l.stream, t, q, which, ch, nch, sx, vj); \
    else launch_pdl(exchange_kernel<RP, BV, false>, grid, 256, 0, l.stream, t, q, which, ch, nch, sx, vj); \
    break;
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

cudaError_t launch_guards(char* base, const uint64_t* offs, int n, uint32_t pattern, unsigned long long* result, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  guards_kernel<<<n, 64, 0, st>>>(base, offs, pattern, result);
  return cudaGetLastError();
}

cudaError_t launch_unpack_codes(const uint8_t* stream, int count, int bits, uint8_t* out, cudaStream_t st) {
  if (count == 0) return cudaSuccess;
  unpack_codes_kernel<<<(count + 255) / 256, 256, 0, st>>>(stream, count, bits, out);
  return cudaGetLastError();
}

cudaError_t launch_scale_reduce(int rp, const Tables& t, int which, float* scales, int n_mat, Launch l) {
  if (n_mat == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP(rp, (launch_pdl(scale_reduce_kernel<RP>, n_mat, 256, 0, l.stream, t, which, scales, n_mat)));
  return cudaGetLastError();
}

cudaError_t launch_sum_dequant(int rp, int which, const Tables& t, const QuantTables& q, const ExchangeChunk* ch,
                               int nch, const SplitExchange& sx, const uint8_t* gathered, int n_streams, Launch l) {
  if (nch == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP(rp, (launch_pdl(sum_dequant_kernel<RP>, nch, 256, 0, l.stream, t, q, which, ch, sx, gathered,
                                    n_streams)));
  return cudaGetLastError();
}

cudaError_t launch_vectors_finish(const VectorJob& vj, Launch l) {
  if (vj.nchunks == 0) return cudaSuccess;
  launch_pdl(vectors_finish_kernel, vj.nchunks, 256, 0, l.stream, vj);
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

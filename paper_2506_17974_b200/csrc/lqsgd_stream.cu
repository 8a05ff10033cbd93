// Bulk-copy (TMA) staged versions of pass 1 and pass 3 (the passes that also write the stream
// back; pass 2 only reads and runs as a high-occupancy register kernel, lqsgd_kernels.cu).  The ring, the copy helpers,
// the geometry of a stage and the bounded waits are in lqsgd_stream_common.cuh.
//
// Each kernel has three roles: a loader warp (fills the ring), 512 consumers, and - where a
// pass writes the streamed data back - a storer warp.  The consumer code of a tile comes in two
// shapes, chosen per tile: "narrow" (a row takes at most 512 threads: one column quad per
// thread, up to 4 or 8 rows per stage) and "wide" (2-3 quads per thread, up to 4 rows).
#include "lqsgd_stream_common.cuh"

namespace lqsgd {
namespace {

template <int RP> struct Shape {
  static constexpr int QPT_WIDE = RP >= 8 ? 1 : (RP == 4 ? 2 : 3);   // quads per thread in wide tiles
  static constexpr int RPT_NARROW = RP >= 8 ? 4 : 8;                  // rows per thread per stage
  static constexpr int RPT_WIDE = 4;
  static constexpr int NRED = RPT_NARROW * RP;                        // widest per-thread set of P sums
};

struct ConsumerState {
  uint32_t it;   // stages consumed so far (ring position)
  int flip;      // alternates per use of the double-buffered reduction / verdict slots
};

// ---------------------------------------------------------------------------------------
// Plain tiles.  A small layer whose rows are not 16-byte aligned (m % 4 != 0: the 64 x 27 first
// convolution) cannot come through the bulk-copy ring.  Rather than pay a kernel launch per pass
// for a few KB, the consumers of the staged kernels take such a layer with ordinary loads while
// the loader already fills the ring for the next tile: a tile is a few whole rows, one warp per
// row, lanes across the columns.  Loader and storer skip these tiles.
// ---------------------------------------------------------------------------------------
template <int RP>
__device__ __forceinline__ void pass1_plain_tile(const Tables& t, const Tile& tl) {
  const LayerDev& L = t.layers[tl.layer];
  const int m = L.m, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float* __restrict__ G = t.grads[(size_t)tl.layer * t.W + tl.worker];
  float* E = L.E + (size_t)tl.worker * L.n * m;
  const float* __restrict__ Qt = L.Qt;
  float* Pp = L.Ppart + (size_t)tl.worker * L.ncc * (size_t)L.n * RP;      // one column chunk: the whole row
  for (int row = tl.row0 + warp; row < tl.row0 + tl.nrows; row += kConsumerWarps) {
    float acc[RP];
#pragma unroll
    for (int j = 0; j < RP; ++j) acc[j] = 0.f;
    for (int c = lane; c < m; c += 32) {
      const size_t off = (size_t)row * m + c;
      const float mv = __ldcs(G + off) + E[off];                             // M = G + E (Eq. 8)
      E[off] = mv;
#pragma unroll
      for (int j = 0; j < RP; ++j) acc[j] = fmaf(mv, __ldg(Qt + (size_t)j * L.mt + c), acc[j]);
    }
#pragma unroll
    for (int j = 0; j < RP; ++j) {
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
      if (lane == 0) Pp[(size_t)row * RP + j] = acc[j];
    }
  }
}

template <int RP>
__device__ __forceinline__ void pass3_plain_tile(const Tables& t, const Tile& tl) {
  const LayerDev& L = t.layers[tl.layer];
  const int m = L.m, W = t.W, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float* __restrict__ Qt = L.Qt;
  const size_t plane = (size_t)L.n * m;
  float* Gh = t.ghat[tl.layer];                                              // may be null
  float* Wt = t.weights ? t.weights[tl.layer] : nullptr;                     // may be null
  for (int row = tl.row0 + warp; row < tl.row0 + tl.nrows; row += kConsumerWarps) {
    float p[RP];
#pragma unroll
    for (int j = 0; j < RP; ++j) p[j] = __ldg(L.Pbar + (size_t)row * RP + j);
    for (int c = lane; c < m; c += 32) {
      const size_t off = (size_t)row * m + c;
      float gh = 0.f;                                                        // G_hat = P_bar Q_bar^T (Eq. 6)
#pragma unroll
      for (int j = 0; j < RP; ++j) gh = fmaf(p[j], __ldg(Qt + (size_t)j * L.mt + c), gh);
      if (Gh) __stcs(Gh + off, gh);
      if (Wt) Wt[off] = fmaf(-t.lr, gh, Wt[off]);                            // model update of Alg. 1
      float* e = L.E + off;
      int w = 0;
      for (; w + 4 <= W; w += 4) {                                           // E_w = M_w - G_hat (Eq. 7)
        float mv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) mv[u] = e[(size_t)(w + u) * plane];
#pragma unroll
        for (int u = 0; u < 4; ++u) e[(size_t)(w + u) * plane] = mv[u] - gh;
      }
      for (; w < W; ++w) e[(size_t)w * plane] -= gh;
    }
  }
}

// ---------------------------------------------------------------------------------------
// pass 1: M = G + E (Eq. 8) over E, partial P = M Q (Alg. 1) per column chunk.
// ---------------------------------------------------------------------------------------
template <int RP, int NST, int QPT, int RPT>
__device__ __forceinline__ bool pass1_consume(const Tables& t, const TileCtx& c, const Ring& ring, float* sG, float* sE,
                                              float* red, volatile int* verdict, ConsumerState& st) {
  constexpr int N = RPT * RP;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const LayerDev& L = t.layers[c.layer];
  const StreamGeo geo = c.geo;
  const Owner o = owner_of(geo, tid);
  float q[QPT * 4 * RP];
  load_q<RP, QPT>(L.Qt, L.mt, c.col0, geo, o, q);
  float* Pp = L.Ppart + (((size_t)c.worker * L.ncc + c.part) * (size_t)c.n + c.row0) * RP;
  const int wpg = geo.tpr >> 5;                // warps per row group
  const int row_f4 = c.ncols >> 2;             // float4 per slab row
  for (int sr = 0; sr < c.nrows; sr += geo.R, ++st.it) {
    const int s = st.it % NST;
    const int rows = min(geo.R, c.nrows - sr);
    const bool ok = mbar_wait(ring.full + s, (st.it / NST) & 1, ring.abort_flag);
    float acc[N];
#pragma unroll
    for (int i = 0; i < N; ++i) acc[i] = 0.f;
    if (ok && o.in_group) {
      const float4* pg = reinterpret_cast<const float4*>(sG + s * kSlab);
      float4* pe = reinterpret_cast<float4*>(sE + s * kSlab);
#pragma unroll
      for (int u = 0; u < RPT; ++u) {
        const int lr = o.g + u * geo.ng;
        if (lr < rows) {
#pragma unroll
          for (int k = 0; k < QPT; ++k) {
            const int quad = o.cq + k * kConsumers;
            if (quad < geo.quads) {
              const int idx = lr * row_f4 + quad;
              const float4 gv = pg[idx];
              const float4 ev = pe[idx];
              const float4 mv = make_float4(gv.x + ev.x, gv.y + ev.y, gv.z + ev.z, gv.w + ev.w);
              pe[idx] = mv;
#pragma unroll
              for (int j = 0; j < RP; ++j) {
                float a = acc[u * RP + j];
                a = fmaf(mv.x, q[(k * 4 + 0) * RP + j], a);
                a = fmaf(mv.y, q[(k * 4 + 1) * RP + j], a);
                a = fmaf(mv.z, q[(k * 4 + 2) * RP + j], a);
                a = fmaf(mv.w, q[(k * 4 + 3) * RP + j], a);
                acc[u * RP + j] = a;
              }
            }
          }
        }
      }
    }
    fence_async_smem();                       // M slab written by this thread -> visible to the bulk store
    __syncwarp();
    if (lane == 0) mbar_arrive(ring.consumed + s);
    warp_transpose_reduce<N, 16>(acc, lane);
    float* rd = red + (st.flip * kConsumerWarps + warp) * Shape<RP>::NRED;
    if constexpr (N >= 32) {
#pragma unroll
      for (int i = 0; i < N / 32; ++i) rd[lane * (N / 32) + i] = acc[i];
    } else {
      if ((lane % (32 / N)) == 0) rd[lane / (32 / N)] = acc[0];
    }
    if (consumers_agree_abort(ring, verdict, st.flip, tid)) {
      if (tid == 0) report_timeout(t, c.layer);
      return false;
    }
    if (tid < rows * RP) {
      const int lr = tid / RP, j = tid - lr * RP;
      const int g2 = lr % geo.ng, u = lr / geo.ng;
      const float* r0 = red + (st.flip * kConsumerWarps + g2 * wpg) * Shape<RP>::NRED + u * RP + j;
      float sum = r0[0];
      for (int w2 = 1; w2 < wpg; ++w2) sum += r0[w2 * Shape<RP>::NRED];   // column segments in order
      Pp[(size_t)(sr + lr) * RP + j] = sum;
    }
    st.flip ^= 1;
  }
  return true;
}

template <int RP, int NST>
__global__ void __launch_bounds__(kThreads, 1)
stream_pass1_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles) {
  prefetch_first_tile(t, tiles, ntiles);
  pdl_wait();
  clear_status_words(t);
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* sG = reinterpret_cast<float*>(smem_raw);
  float* sE = sG + NST * kSlab;
  float* red = sE + NST * kSlab;                              // [2][16 warps][NRED]
  uint64_t* bars = reinterpret_cast<uint64_t*>(red + 2 * kConsumerWarps * Shape<RP>::NRED);
  volatile int* flags = reinterpret_cast<volatile int*>(bars + 3 * NST);   // abort, wait limit, verdict[2]
  const Ring ring{bars, bars + NST, bars + 2 * NST, flags};
  ring_init(ring, NST, true, t.wait_limit);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (warp == kConsumerWarps) {                 // ---- loader
    const uint64_t pol_first = policy_evict_first();
    bool ok = true;
    int last_layer = 0;
    uint32_t it = 0;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      if (tiles[ti].pad) continue;              // plain tile: the consumers fetch it themselves
      const TileCtx c = tile_ctx<RP>(t, tiles[ti]);
      last_layer = c.layer;
      const float* G = t.grads[(size_t)c.layer * t.W + c.worker] + (size_t)c.row0 * c.m + c.col0;
      const float* E = t.layers[c.layer].E + ((size_t)c.worker * c.n + c.row0) * c.m + c.col0;
      for (int sr = 0; sr < c.nrows; sr += c.geo.R, ++it) {
        const int s = it % NST;
        const uint32_t k = it / NST;
        const int rows = min(c.geo.R, c.nrows - sr);
        if (k > 0) ok = warp_wait(ring.empty + s, (k - 1) & 1, ring.abort_flag, lane);
        if (!ok) break;
        if (test_skips_stage(t, 1, it)) continue;     // test support: this stage's copies are left out, its waiters give up
        if (lane == 0) mbar_arrive_expect_tx(ring.full + s, 2u * rows * c.ncols * 4u);
        __syncwarp();
        load_slab(sG + s * kSlab, G, c, sr, rows, ring.full + s, lane, pol_first);
        load_slab(sE + s * kSlab, E, c, sr, rows, ring.full + s, lane, pol_first);
      }
    }
    if (!ok && lane == 0) { report_timeout(t, last_layer); loader_drain<NST>(ring, it); }
    return;
  }
  if (warp == kConsumerWarps + 1) {             // ---- storer: M slabs back over E
    const uint64_t pol_last = policy_evict_last();
    bool ok = true;
    uint32_t it = 0;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      if (tiles[ti].pad) continue;
      const TileCtx c = tile_ctx<RP>(t, tiles[ti]);
      float* E = t.layers[c.layer].E + ((size_t)c.worker * c.n + c.row0) * c.m + c.col0;
      for (int sr = 0; sr < c.nrows; sr += c.geo.R, ++it) {
        const int s = it % NST;
        const int rows = min(c.geo.R, c.nrows - sr);
        ok = warp_wait(ring.consumed + s, (it / NST) & 1, ring.abort_flag, lane);
        if (!ok) break;
        store_slab(E, sE + s * kSlab, c, sr, rows, lane, pol_last);     // pass 2 starts on the M written last
        bulk_commit();
        bulk_wait_read0();
        __syncwarp();
        if (lane == 0) mbar_arrive(ring.empty + s);
      }
    }
    bulk_wait_all0();
    return;
  }
  ConsumerState st{0, 0};
  for (int ti = blockIdx.x; ti < ntiles; ti += gridDim.x) {
    if (tiles[ti].pad) { pass1_plain_tile<RP>(t, tiles[ti]); continue; }
    const TileCtx c = tile_ctx<RP>(t, tiles[ti]);
    bool ok;
    if (c.geo.qpt == 1) ok = pass1_consume<RP, NST, 1, Shape<RP>::RPT_NARROW>(t, c, ring, sG, sE, red, flags + 2, st);
    else ok = pass1_consume<RP, NST, Shape<RP>::QPT_WIDE, Shape<RP>::RPT_WIDE>(t, c, ring, sG, sE, red, flags + 2, st);
    if (!ok) return;
  }
}

// ---------------------------------------------------------------------------------------
// pass 3: G_hat = P_bar Q_bar^T (Eq. 6), E_w = M_w - G_hat (Eq. 7).  For every block of R rows
// the workers' M slabs follow one another through the ring; G_hat of the block is formed once
// (before waiting for the first worker's slab) and kept in registers.
// ---------------------------------------------------------------------------------------
template <int RP, int NST, int QPT, int RPT>
__device__ __forceinline__ bool pass3_consume(const Tables& t, const TileCtx& c, const Ring& ring, float* sM, float* pb_warp,
                                              uint32_t& it) {
  const int tid = threadIdx.x, lane = tid & 31;
  const LayerDev& L = t.layers[c.layer];
  const StreamGeo geo = c.geo;
  const Owner o = owner_of(geo, tid);
  const float* __restrict__ Pbar = L.Pbar;
  const int row_f4 = c.ncols >> 2, m = c.m, W = t.W;
  float q[QPT * 4 * RP];
  load_q<RP, QPT>(L.Qt, L.mt, c.col0, geo, o, q);
  float* Gh0 = t.ghat[c.layer];                                            // may be null
  float* Wt0 = t.weights ? t.weights[c.layer] : nullptr;                   // may be null
  float* Gh = Gh0 ? Gh0 + (size_t)c.row0 * m + c.col0 : nullptr;
  float* Wt = Wt0 ? Wt0 + (size_t)c.row0 * m + c.col0 : nullptr;
  const float step = t.lr;
  // The block's rows of P_bar (RPT rows of RP floats, the same for the whole warp: at most 32 floats) are fetched
  // one float per lane, as soon as the previous block's last slab has been handed on, and passed round through the
  // warp's 128 bytes of shared memory: one load per warp and block instead of eight per thread.  (Fetching a whole
  // block ahead, under the previous block's slabs, is faster still on narrow layers and up to 9 % slower on
  // matrices of a gigabyte, where the pass runs at the memory's speed and the consumers' pace matters: not kept.)
  auto fetch_pbar = [&](int sr) -> float {
    const int u = lane / RP, lr = o.g + u * geo.ng;
    const bool want = lane < RPT * RP && o.in_group && lr < min(geo.R, c.nrows - sr);
    return want ? __ldg(Pbar + (size_t)(c.row0 + sr + lr) * RP + (lane % RP)) : 0.f;
  };
  float pnext = fetch_pbar(0);
  for (int sr = 0; sr < c.nrows; sr += geo.R) {
    const int rows = min(geo.R, c.nrows - sr);
    float4 gh[RPT * QPT];
    {
      float p[RPT * RP];
      pb_warp[lane] = pnext;
      __syncwarp();
#pragma unroll
      for (int i = 0; i < RPT * RP; i += (RP % 4 == 0 ? 4 : RP)) {
        if constexpr (RP % 4 == 0) {
          const float4 v = *reinterpret_cast<const float4*>(pb_warp + i);
          p[i] = v.x; p[i + 1] = v.y; p[i + 2] = v.z; p[i + 3] = v.w;
        } else if constexpr (RP == 2) {
          const float2 v = *reinterpret_cast<const float2*>(pb_warp + i);
          p[i] = v.x; p[i + 1] = v.y;
        } else {
          p[i] = pb_warp[i];
        }
      }
#pragma unroll
      for (int u = 0; u < RPT; ++u) {
        const int lr = o.g + u * geo.ng;
#pragma unroll
        for (int k = 0; k < QPT; ++k) {
          float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
          for (int j = 0; j < RP; ++j) {
            const float pj = p[u * RP + j];
            a0 = fmaf(pj, q[(k * 4 + 0) * RP + j], a0);
            a1 = fmaf(pj, q[(k * 4 + 1) * RP + j], a1);
            a2 = fmaf(pj, q[(k * 4 + 2) * RP + j], a2);
            a3 = fmaf(pj, q[(k * 4 + 3) * RP + j], a3);
          }
          gh[u * QPT + k] = make_float4(a0, a1, a2, a3);
          const int quad = o.cq + k * kConsumers;
          if (o.in_group && lr < rows && quad < geo.quads) {
            const float4 g4 = gh[u * QPT + k];
            if (Gh) __stcs(reinterpret_cast<float4*>(Gh + (size_t)(sr + lr) * m) + quad, g4);
            if (Wt) {                              // model update of Alg. 1: w <- w - lr * G_hat
              float4* wp = reinterpret_cast<float4*>(Wt + (size_t)(sr + lr) * m) + quad;
              float4 wv = __ldcs(wp);
              wv.x = fmaf(-step, g4.x, wv.x); wv.y = fmaf(-step, g4.y, wv.y);
              wv.z = fmaf(-step, g4.z, wv.z); wv.w = fmaf(-step, g4.w, wv.w);
              __stcs(wp, wv);
            }
          }
        }
      }
    }
    for (int w = 0; w < W; ++w, ++it) {
      const int s = it % NST;
      const bool ok = mbar_wait(ring.full + s, (it / NST) & 1, ring.abort_flag);
      if (ok && o.in_group) {
        float4* pm = reinterpret_cast<float4*>(sM + s * kSlab);
#pragma unroll
        for (int u = 0; u < RPT; ++u) {
          const int lr = o.g + u * geo.ng;
          if (lr < rows) {
#pragma unroll
            for (int k = 0; k < QPT; ++k) {
              const int quad = o.cq + k * kConsumers;
              if (quad < geo.quads) {
                const int idx = lr * row_f4 + quad;
                const float4 mv = pm[idx];
                const float4 g4 = gh[u * QPT + k];
                pm[idx] = make_float4(mv.x - g4.x, mv.y - g4.y, mv.z - g4.z, mv.w - g4.w);
              }
            }
          }
        }
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(ring.consumed + s);
    }
    if (sr + geo.R < c.nrows) pnext = fetch_pbar(sr + geo.R);
  }
  if (*ring.abort_flag) {                      // no common barrier in this pass: each consumer leaves on its own
    if (tid == 0) report_timeout(t, c.layer);
    return false;
  }
  return true;
}

template <int RP, int NST>
__global__ void __launch_bounds__(kThreads, 1)
stream_pass3_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles) {
  prefetch_first_tile(t, tiles, ntiles);
  pdl_wait();
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* sM = reinterpret_cast<float*>(smem_raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sM + NST * kSlab);
  volatile int* flags = reinterpret_cast<volatile int*>(bars + 3 * NST);   // abort, wait limit
  const Ring ring{bars, bars + NST, bars + 2 * NST, flags};
  __shared__ __align__(16) float pb_rows[kConsumerWarps][32];     // a block's rows of P_bar, per consumer warp
  ring_init(ring, NST, true, t.wait_limit);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int W = t.W;

  if (warp == kConsumerWarps) {                 // ---- loader
    const uint64_t pol_first = policy_evict_first();
    bool ok = true;
    int last_layer = 0;
    uint32_t it = 0;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      if (tiles[ti].pad) continue;
      const TileCtx c = tile_ctx<RP>(t, tiles[ti]);
      last_layer = c.layer;
      const size_t plane = (size_t)c.n * c.m;
      const float* M0 = t.layers[c.layer].E + (size_t)c.row0 * c.m + c.col0;
      for (int sr = 0; sr < c.nrows && ok; sr += c.geo.R) {
        const int rows = min(c.geo.R, c.nrows - sr);
        for (int w = 0; w < W; ++w, ++it) {
          const int s = it % NST;
          const uint32_t k = it / NST;
          if (k > 0) ok = warp_wait(ring.empty + s, (k - 1) & 1, ring.abort_flag, lane);
          if (!ok) break;
          if (test_skips_stage(t, 3, it)) continue;   // test support, as in pass 1
          if (lane == 0) mbar_arrive_expect_tx(ring.full + s, (uint32_t)rows * c.ncols * 4u);
          __syncwarp();
          load_slab(sM + s * kSlab, M0 + (size_t)w * plane, c, sr, rows, ring.full + s, lane, pol_first);
        }
      }
    }
    if (!ok && lane == 0) { report_timeout(t, last_layer); loader_drain<NST>(ring, it); }
    return;
  }
  if (warp == kConsumerWarps + 1) {             // ---- storer: E slabs
    const uint64_t pol_first = policy_evict_first();
    bool ok = true;
    uint32_t it = 0;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      if (tiles[ti].pad) continue;
      const TileCtx c = tile_ctx<RP>(t, tiles[ti]);
      const size_t plane = (size_t)c.n * c.m;
      float* E0 = t.layers[c.layer].E + (size_t)c.row0 * c.m + c.col0;
      for (int sr = 0; sr < c.nrows && ok; sr += c.geo.R) {
        const int rows = min(c.geo.R, c.nrows - sr);
        for (int w = 0; w < W; ++w, ++it) {
          const int s = it % NST;
          ok = warp_wait(ring.consumed + s, (it / NST) & 1, ring.abort_flag, lane);
          if (!ok) break;
          store_slab(E0 + (size_t)w * plane, sM + s * kSlab, c, sr, rows, lane, pol_first);
          bulk_commit();
          bulk_wait_read0();
          __syncwarp();
          if (lane == 0) mbar_arrive(ring.empty + s);
        }
      }
    }
    bulk_wait_all0();
    return;
  }
  uint32_t it = 0;
  for (int ti = blockIdx.x; ti < ntiles; ti += gridDim.x) {
    if (tiles[ti].pad) { pass3_plain_tile<RP>(t, tiles[ti]); continue; }
    const TileCtx c = tile_ctx<RP>(t, tiles[ti]);
    bool ok;
    if (c.geo.qpt == 1) ok = pass3_consume<RP, NST, 1, Shape<RP>::RPT_NARROW>(t, c, ring, sM, pb_rows[warp], it);
    else ok = pass3_consume<RP, NST, Shape<RP>::QPT_WIDE, Shape<RP>::RPT_WIDE>(t, c, ring, sM, pb_rows[warp], it);
    if (!ok) return;
  }
}

size_t smem_pass1(int RP, int NST) {
  const int nred = (RP >= 8 ? 4 : 8) * RP;
  return (size_t)NST * 2 * kSlab * 4 + 2 * kConsumerWarps * nred * 4 + (3 * NST + 2) * 8;
}
size_t smem_pass3(int /*RP*/, int NST) { return (size_t)NST * kSlab * 4 + (3 * NST + 2) * 8; }

template <typename K>
cudaError_t launch_staged(K kernel, size_t smem, const Tables& t, const Tile* tiles, int ntiles, Launch l) {
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  launch_pdl(kernel, l.grid, kThreads, smem, l.stream, t, tiles, ntiles);
  return cudaGetLastError();
}

}  // namespace

#define LQSGD_DISPATCH_RP8(RPV, ...)                        \
  switch (RPV) {                                            \
    case 1: { constexpr int RP = 1; __VA_ARGS__; } break;   \
    case 2: { constexpr int RP = 2; __VA_ARGS__; } break;   \
    case 4: { constexpr int RP = 4; __VA_ARGS__; } break;   \
    case 8: { constexpr int RP = 8; __VA_ARGS__; } break;   \
    default: return cudaErrorInvalidValue;                  \
  }

constexpr int kNst1 = 3, kNst3 = 4;   // pass 3: a ring of 4 slabs; with 5 the loads ran further ahead than the memory likes on matrices of a gigabyte

cudaError_t launch_stream_pass1(int rp, const Tables& t, const Tile* tiles, int ntiles, Launch l) {
  if (ntiles == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP8(rp, return launch_staged(stream_pass1_kernel<RP, kNst1>, smem_pass1(RP, kNst1), t, tiles, ntiles, l));
  return cudaSuccess;
}
cudaError_t launch_stream_pass3(int rp, const Tables& t, const Tile* tiles, int ntiles, Launch l) {
  if (ntiles == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP8(rp, return launch_staged(stream_pass3_kernel<RP, kNst3>, smem_pass3(RP, kNst3), t, tiles, ntiles, l));
  return cudaSuccess;
}

}  // namespace lqsgd

// The whole LQ-SGD round (Algorithm 1, loop body) in ONE launch, for gradient sets small enough that
// M = G + E of every layer and worker fits in the shared memory of the GPU's SMs together.
//
// A round over a small set is not bound by HBM but by its chain of dependent steps: pass 1, Gram, Cholesky
// and solve, exchange of P, pass 2, reduction of Q_w, exchange of Q, pass 3.  As separate kernels every arrow
// of that chain costs a launch boundary, and M makes three trips through memory.  Here one cooperative grid
// (one CTA per SM, all co-resident) walks the chain with grid barriers between the steps, and every CTA keeps
// its tiles of M in shared memory from pass 1 to pass 3:
//
//   A  pass 1   E tiles arrive by bulk copy straight into their resident place, G streams through registers;
//               M = G + E (Eq. 8) replaces E in shared memory; partial P = M Q per column chunk
//   B  Orthonormalize (one CTA per small layer and worker; Gram blocks for tall layers), the 1-D tensors' mean
//   B2 tall layers only: Cholesky + solve per block of rows
//   D  every CTA forms P_bar of its own tiles' rows itself (scale, LogQuantize, exact integer worker sum,
//      LogDequantize: Eq. 4, Eq. 1, Eq. 5) and goes straight on to pass 2, partial Q = M^T P_bar from the
//      resident tiles
//   E  Q_w = fixed-order sum of the partials, block maxima; beside it, on other CTAs, the exchange of P proper
//      (codes packed into the payloads, P_bar stored): nothing before pass 3 waits for it
//   G  likewise Q_bar of the tile's columns, then pass 3: G_hat = P_bar Q_bar^T (Eq. 6), E = M - G_hat (Eq. 7)
//      in place, tiles go back by bulk store; afterwards the exchange of Q proper (payloads, Q for the next round)
//
// HBM traffic falls from 24 + 4/W to 12 + 4/W bytes per worker-element (G and E in, E and G_hat out), seven
// launches become one, and the chain is four grid barriers long (five with tall layers).  The steps between the
// passes are the device functions the multi-kernel round uses (lqsgd_factor.cuh), reading through L2 what other
// CTAs wrote before the barrier.
//
// Grid barrier.  Counters in global memory, one per barrier of a launch, in two sets that alternate between
// launches (a launch clears the other set, so nothing has to be reset between two rounds and a graph replay
// works).  A CTA arrives with a release, polls with an acquire, and gives up after a bounded number of polls:
// then the layer-0 status word gets LQSGD_STATUS_TIMEOUT, the CTA waits for its own copies in flight and
// returns.  The cooperative launch guarantees that all CTAs are resident, so in normal operation no CTA waits
// for one that is not running.
#include "lqsgd_factor.cuh"
#include "lqsgd_stream_common.cuh"

namespace lqsgd {
namespace {

constexpr int kResWarps = kResThreads / 32;
constexpr uint32_t kGridPollLimit = 1u << 21;     // polls of ~0.5 us: about a second
constexpr int kResControlBytes = 2048;            // barriers, flags, the local exchange's tables

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t v;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(v));
  return v;
}
__device__ __forceinline__ void red_release_add(uint32_t* p, uint32_t v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

template <int A, int B2> struct CMax { static constexpr int value = A > B2 ? A : B2; };

// Scratch shared memory the steps between the passes and the passes' own reductions need at this padded rank.
template <int RP> struct ResScratch {
  static constexpr int kPb = kResMaxTileRows * RP * 4;                       // a tile's rows of P_bar
  static constexpr int kRed = (kResThreads / 2) * 4 * RP * 4;                // pass 2: half the threads hand 4 RP sums over
  static constexpr int kRed1 = 2 * kResWarps * 8 * RP * 4;                   // pass 1: two buffers of per-warp sums
  static constexpr int kPass = kPb + CMax<kRed, kRed1>::value;
  static constexpr int kBodies = CMax<CMax<(int)sizeof(OrthSmallSmem<RP>), (int)sizeof(ApplySmem<RP, kResThreads>)>::value,
                                      CMax<CMax<(int)sizeof(ReduceGramSmem<RP>), (int)sizeof(QReduceSmem<RP, kResThreads>)>::value,
                                           (int)sizeof(ExchangeSmem<RP, kResThreads>)>::value>::value;
  static constexpr int value = (CMax<kPass, kBodies>::value + 127) / 128 * 128;
};

struct ResGeo {
  int quads, tpr, ng, rpt, R;
};
template <int RP>
__device__ __forceinline__ ResGeo res_geo(int ncols) {
  ResGeo g;
  g.quads = ncols >> 2;
  g.tpr = (g.quads + 31) & ~31;
  g.ng = kResThreads / g.tpr;
  g.rpt = RP >= 8 ? 4 : 8;
  g.R = g.ng * g.rpt;
  return g;
}

struct ResShared {
  uint64_t tile_bar[kResMaxTiles];     // E tile landed
  volatile int wait_ctl[2];            // abort flag, limit of the mbarrier waits (see lqsgd_stream_common.cuh)
  volatile int sync_ok;                // outcome of the last grid barrier, for the whole CTA
  uint32_t slot;                       // which of the two counter sets this launch uses
};

// ---------------------------------------------------------------------------------------
// Grid barrier number k of this launch.  Returns false (to every thread alike) when the wait ran out.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ bool grid_barrier(const ResidentArgs& a, const Tables& t, ResShared& sh, int k) {
  __syncthreads();       // the CTA's writes are ordered before thread 0's release below
  if (threadIdx.x == 0) {
    uint32_t* ctr = a.sync + 1 + sh.slot * kResBarriers + k;
    const uint32_t limit = t.wait_limit ? t.wait_limit : kGridPollLimit;
    // test support: CTA 0 stays away from barrier number test_skip_stage, so every wait on it runs out
    const bool stay_away = t.test_skip_pass == 4 && blockIdx.x == 0 && k == t.test_skip_stage;
    if (!stay_away) red_release_add(ctr, 1u);
    int ok = 1;
    uint32_t polls = 0;
    while (ld_acquire_u32(ctr) < gridDim.x) {
      if (++polls >= limit) { ok = 0; break; }
    }
    sh.sync_ok = ok;
  }
  __syncthreads();       // and thread 0's acquire before everything the CTA reads afterwards
  return sh.sync_ok != 0;
}

// ---------------------------------------------------------------------------------------
// pass 1 of one resident tile.  Thread = (row group g, column quad cq) as in the staged passes; a stage is R rows.
// ---------------------------------------------------------------------------------------
template <int RP>
__device__ __forceinline__ bool res_pass1_tile(const Tables& t, const ResTile& tl, float* tile, uint64_t* bar, float* red,
                                               ResShared& sh) {
  constexpr int RPT = RP >= 8 ? 4 : 8;
  constexpr int N = RPT * RP;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const LayerDev& L = t.layers[tl.layer];
  const int m = L.m;
  const ResGeo geo = res_geo<RP>(tl.ncols);
  const int g = tid / geo.tpr, cq = tid - g * geo.tpr;
  const bool active = g < geo.ng && cq < geo.quads;
  const int wpg = geo.tpr >> 5, row_f4 = tl.ncols >> 2;
  float q[4 * RP];
#pragma unroll
  for (int j = 0; j < RP; ++j) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (active) v = __ldcg(reinterpret_cast<const float4*>(L.Qt + (size_t)j * L.mt + tl.col0) + cq);
    q[0 * RP + j] = v.x; q[1 * RP + j] = v.y; q[2 * RP + j] = v.z; q[3 * RP + j] = v.w;
  }
  const float4* G4 = reinterpret_cast<const float4*>(t.grads[(size_t)tl.layer * t.W + tl.worker] + (size_t)tl.row0 * m + tl.col0) + cq;
  const int m4 = m >> 2;
  float4 gv[RPT];
  auto fetch = [&](int sr, float4(&dst)[RPT]) {
#pragma unroll
    for (int u = 0; u < RPT; ++u) {
      const int lr = sr + g + u * geo.ng;
      dst[u] = (active && lr < tl.nrows) ? __ldcs(G4 + (size_t)lr * m4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  fetch(0, gv);
  const bool landed = mbar_wait(bar, 0, sh.wait_ctl);          // the tile's E, by bulk copy
  if (__syncthreads_or(landed ? 0 : 1)) return false;
  float4* tile4 = reinterpret_cast<float4*>(tile);
  float* Pp = L.Ppart + (((size_t)tl.worker * L.ncc + tl.part_c) * (size_t)L.n + tl.row0) * RP;
  int flip = 0;
  for (int sr = 0; sr < tl.nrows; sr += geo.R) {
    const int rows = min(geo.R, tl.nrows - sr);
    float4 gn[RPT];
    if (sr + geo.R < tl.nrows) fetch(sr + geo.R, gn);
    float acc[N];
#pragma unroll
    for (int i = 0; i < N; ++i) acc[i] = 0.f;
    if (active) {
#pragma unroll
      for (int u = 0; u < RPT; ++u) {
        const int lr = sr + g + u * geo.ng;
        if (lr < tl.nrows) {
          const int idx = lr * row_f4 + cq;
          const float4 ev = tile4[idx];
          const float4 mv = make_float4(gv[u].x + ev.x, gv[u].y + ev.y, gv[u].z + ev.z, gv[u].w + ev.w);
          tile4[idx] = mv;                                      // M = G + E (Eq. 8), kept until pass 3
#pragma unroll
          for (int j = 0; j < RP; ++j) {
            float s = acc[u * RP + j];
            s = fmaf(mv.x, q[0 * RP + j], s);
            s = fmaf(mv.y, q[1 * RP + j], s);
            s = fmaf(mv.z, q[2 * RP + j], s);
            s = fmaf(mv.w, q[3 * RP + j], s);
            acc[u * RP + j] = s;
          }
        }
      }
    }
    warp_transpose_reduce<N, 16>(acc, lane);
    float* rd = red + (flip * kResWarps + warp) * (8 * RP);
    if constexpr (N >= 32) {
#pragma unroll
      for (int i = 0; i < N / 32; ++i) rd[lane * (N / 32) + i] = acc[i];
    } else {
      if ((lane % (32 / N)) == 0) rd[lane / (32 / N)] = acc[0];
    }
    __syncthreads();
    if (tid < rows * RP) {
      const int lr = tid / RP, j = tid - lr * RP;
      const int g2 = lr % geo.ng, u = lr / geo.ng;
      const float* r0 = red + (flip * kResWarps + g2 * wpg) * (8 * RP) + u * RP + j;
      float sum = r0[0];
      for (int w2 = 1; w2 < wpg; ++w2) sum += r0[w2 * (8 * RP)];     // column segments in order
      Pp[(size_t)(sr + lr) * RP + j] = sum;
    }
    flip ^= 1;
#pragma unroll
    for (int u = 0; u < RPT; ++u) gv[u] = gn[u];
  }
  return true;
}

// A tile of a layer whose rows are not 16-byte aligned: whole rows, ordinary loads, one warp per row.
template <int RP>
__device__ __noinline__ void res_pass1_plain(const Tables& t, const ResTile& tl, float* tile) {
  const LayerDev& L = t.layers[tl.layer];
  const int m = L.m, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float* __restrict__ G = t.grads[(size_t)tl.layer * t.W + tl.worker] + (size_t)tl.row0 * m;
  const float* E = L.E + ((size_t)tl.worker * L.n + tl.row0) * m;
  float* Pp = L.Ppart + ((size_t)tl.worker * L.ncc * L.n + tl.row0) * RP;
  for (int row = warp; row < tl.nrows; row += kResWarps) {
    float acc[RP];
#pragma unroll
    for (int j = 0; j < RP; ++j) acc[j] = 0.f;
    for (int c = lane; c < m; c += 32) {
      const float mv = __ldcs(G + (size_t)row * m + c) + __ldcs(E + (size_t)row * m + c);
      tile[row * m + c] = mv;
#pragma unroll
      for (int j = 0; j < RP; ++j) acc[j] = fmaf(mv, __ldcg(L.Qt + (size_t)j * L.mt + c), acc[j]);
    }
#pragma unroll
    for (int j = 0; j < RP; ++j) {
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
      if (lane == 0) Pp[(size_t)row * RP + j] = acc[j];
    }
  }
}

// The tile's rows of P_bar, from L2 into scratch.
template <int RP>
__device__ __forceinline__ void res_load_pbar(const LayerDev& L, const ResTile& tl, float* pb) {
  const float* src = L.Pbar + (size_t)tl.row0 * RP;
  for (int i = threadIdx.x; i < tl.nrows * RP; i += kResThreads) pb[i] = __ldcg(src + i);
}

// ---------------------------------------------------------------------------------------
// pass 2 of one resident tile: partial Q[col][:] = sum over the tile's rows of M[row][col] P_bar[row][:], with the
// tile's rows of P_bar in pb (shared memory).  Row groups are summed pairwise through scratch in a fixed order.
// ---------------------------------------------------------------------------------------
template <int RP>
__device__ __forceinline__ void res_pass2_tile(const Tables& t, const ResTile& tl, const float* tile, const float* pb, float* red) {
  const int tid = threadIdx.x;
  const LayerDev& L = t.layers[tl.layer];
  float* Qp = L.Qpart + (((size_t)tl.worker * L.nrb + tl.part_r) * (size_t)L.m) * RP;
  if (tl.plain) {
    const int m = L.m;
    for (int c = tid; c < m; c += kResThreads) {
      float acc[RP];
#pragma unroll
      for (int j = 0; j < RP; ++j) acc[j] = 0.f;
      for (int row = 0; row < tl.nrows; ++row) {
        const float mv = tile[row * m + c];
#pragma unroll
        for (int j = 0; j < RP; ++j) acc[j] = fmaf(mv, pb[row * RP + j], acc[j]);
      }
      store_contig<RP>(Qp + (size_t)c * RP, acc);
    }
    __syncthreads();
    return;
  }
  const ResGeo geo = res_geo<RP>(tl.ncols);
  const int g = tid / geo.tpr, cq = tid - g * geo.tpr;
  const bool active = g < geo.ng && cq < geo.quads;
  const int row_f4 = tl.ncols >> 2;
  const float4* tile4 = reinterpret_cast<const float4*>(tile);
  float acc[4 * RP];
#pragma unroll
  for (int i = 0; i < 4 * RP; ++i) acc[i] = 0.f;
  if (active) {
    for (int lr = g; lr < tl.nrows; lr += geo.ng) {
      const float4 mv = tile4[lr * row_f4 + cq];
      float p[RP];
#pragma unroll
      for (int j = 0; j < RP; ++j) p[j] = pb[lr * RP + j];
#pragma unroll
      for (int j = 0; j < RP; ++j) {
        acc[0 * RP + j] = fmaf(mv.x, p[j], acc[0 * RP + j]);
        acc[1 * RP + j] = fmaf(mv.y, p[j], acc[1 * RP + j]);
        acc[2 * RP + j] = fmaf(mv.z, p[j], acc[2 * RP + j]);
        acc[3 * RP + j] = fmaf(mv.w, p[j], acc[3 * RP + j]);
      }
    }
  }
  int top = 1;
  while (top < geo.ng) top <<= 1;
  for (int s = top >> 1; s >= 1; s >>= 1) {               // groups [s, 2s) hand their sums to groups [0, s)
    if (active && g >= s && g < 2 * s) {
      float* dst = red + (size_t)(g - s) * geo.tpr * (4 * RP) + cq;
#pragma unroll
      for (int k = 0; k < 4 * RP; ++k) dst[k * geo.tpr] = acc[k];
    }
    __syncthreads();
    if (active && g < s && g + s < geo.ng) {
      const float* srcp = red + (size_t)g * geo.tpr * (4 * RP) + cq;
#pragma unroll
      for (int k = 0; k < 4 * RP; ++k) acc[k] += srcp[k * geo.tpr];
    }
    __syncthreads();
  }
  if (active && g == 0) store_contig<4 * RP>(Qp + (size_t)(tl.col0 + 4 * cq) * RP, acc);
  __syncthreads();                                          // pb and red are reused by the next tile
}

// ---------------------------------------------------------------------------------------
// pass 3 of one resident tile, with Q_bar of the tile's columns in qb (shared memory, [ncols][RP]):
// G_hat = P_bar Q_bar^T (Eq. 6), E = M - G_hat (Eq. 7) in place; the tile holding
// worker 0's copy of a region also writes G_hat and applies the model update.  Returns with the tile's E in
// shared memory, visible to the bulk-copy engine.
// ---------------------------------------------------------------------------------------
template <int RP>
__device__ __forceinline__ void res_pass3_tile(const Tables& t, const ResTile& tl, float* tile, float* pb, const float* qb) {
  const int tid = threadIdx.x;
  const LayerDev& L = t.layers[tl.layer];
  const int m = L.m;
  res_load_pbar<RP>(L, tl, pb);
  __syncthreads();
  float* Gh = (tl.writes_ghat && t.ghat[tl.layer]) ? t.ghat[tl.layer] + (size_t)tl.row0 * m + tl.col0 : nullptr;
  float* Wt = (tl.writes_ghat && t.weights && t.weights[tl.layer]) ? t.weights[tl.layer] + (size_t)tl.row0 * m + tl.col0 : nullptr;
  const float step = t.lr;
  if (tl.plain) {
    float* Eg = L.E + ((size_t)tl.worker * L.n + tl.row0) * m;
    for (int idx = tid; idx < tl.nrows * m; idx += kResThreads) {
      const int row = idx / m, c = idx - row * m;
      float gh = 0.f;
#pragma unroll
      for (int j = 0; j < RP; ++j) gh = fmaf(pb[row * RP + j], qb[c * RP + j], gh);
      Eg[idx] = tile[idx] - gh;
      if (Gh) __stcs(Gh + idx, gh);
      if (Wt) Wt[idx] = fmaf(-step, gh, Wt[idx]);
    }
    __syncthreads();
    return;
  }
  const ResGeo geo = res_geo<RP>(tl.ncols);
  const int g = tid / geo.tpr, cq = tid - g * geo.tpr;
  const bool active = g < geo.ng && cq < geo.quads;
  const int row_f4 = tl.ncols >> 2, m4 = m >> 2;
  if (active) {
    float q[4 * RP];                                          // Q_bar of this round, rows 4 cq .. 4 cq + 3 of the tile's columns
#pragma unroll
    for (int i = 0; i < 4 * RP; ++i) q[i] = qb[4 * cq * RP + i];
    float4* tile4 = reinterpret_cast<float4*>(tile);
    for (int lr = g; lr < tl.nrows; lr += geo.ng) {
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
      for (int j = 0; j < RP; ++j) {
        const float pj = pb[lr * RP + j];
        a0 = fmaf(pj, q[0 * RP + j], a0);
        a1 = fmaf(pj, q[1 * RP + j], a1);
        a2 = fmaf(pj, q[2 * RP + j], a2);
        a3 = fmaf(pj, q[3 * RP + j], a3);
      }
      const int idx = lr * row_f4 + cq;
      const float4 mv = tile4[idx];
      tile4[idx] = make_float4(mv.x - a0, mv.y - a1, mv.z - a2, mv.w - a3);
      if (Gh) __stcs(reinterpret_cast<float4*>(Gh) + (size_t)lr * m4 + cq, make_float4(a0, a1, a2, a3));
      if (Wt) {
        float4* wp = reinterpret_cast<float4*>(Wt) + (size_t)lr * m4 + cq;
        float4 wv = __ldcs(wp);
        wv.x = fmaf(-step, a0, wv.x); wv.y = fmaf(-step, a1, wv.y);
        wv.z = fmaf(-step, a2, wv.z); wv.w = fmaf(-step, a3, wv.w);
        __stcs(wp, wv);
      }
    }
  }
  fence_async_smem();                                       // the bulk store reads what was just written
  __syncthreads();
}

// Each step as a real function: one copy of its code, fetched only if it runs.  The round goes through every
// step once per launch from a cold instruction cache, and fetching code is a large part of what a step costs.
template <int RP> __device__ __noinline__ void step_orth_small(const Tables& t, const FactorBlock fb, void* scratch) {
  p_orth_small_body<RP, true>(t, fb, threadIdx.x, scratch);
}
template <int RP> __device__ __noinline__ void step_reduce_gram(const Tables& t, const FactorBlock fb, void* scratch) {
  p_reduce_gram_body<RP, kResThreads, true>(t, fb, threadIdx.x, scratch);
}
template <int RP> __device__ __noinline__ void step_apply(const Tables& t, const FactorBlock fb, void* scratch) {
  p_apply_body<RP, kResThreads, true>(t, fb, threadIdx.x, scratch);
}
template <int RP> __device__ __noinline__ void step_q_reduce(const Tables& t, const FactorBlock fb, void* scratch) {
  q_reduce_body<RP, kResThreads, true>(t, fb, threadIdx.x, scratch);
}
template <int RP> __device__ __noinline__ void step_exchange(const Tables& t, const QuantTables& qt, int which, const ExchangeChunk ch,
                                                             void* scratch) {
  SplitExchange sx{};
  exchange_body<RP, 0, kResThreads, true>(t, qt, which, ch, sx, threadIdx.x, scratch);
}
__device__ __noinline__ void step_vectors(const VectorJob& vj, int job, uint8_t* payload, uint64_t payload_stride, int W) {
  vectors_block(vj, job, threadIdx.x, payload, payload_stride, W);
}

template <int RP>
__global__ void __launch_bounds__(kResThreads, 1)
resident_round_kernel(Tables t, ResidentArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* scratch = smem_raw;
  ResShared& sh = *reinterpret_cast<ResShared*>(smem_raw + ResScratch<RP>::value);
  void* xl = smem_raw + ResScratch<RP>::value + 256;          // scale and thresholds of a CTA's own exchange
  float* resident = reinterpret_cast<float*>(smem_raw + ResScratch<RP>::value + kResControlBytes);
  static_assert(sizeof(ResShared) <= 256 && 256 + sizeof(ExchangeLocalSmem<RP, kResThreads>) <= kResControlBytes, "control block");
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int t_begin = a.cta_begin[blockIdx.x], t_end = a.cta_begin[blockIdx.x + 1];

  if (tid == 0) {
    for (int i = 0; i < kResMaxTiles; ++i) mbar_init(sh.tile_bar + i, 1);
    wait_ctl_init(sh.wait_ctl, t.wait_limit);
    sh.sync_ok = 1;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  clear_status_words(t);
  __syncthreads();
  // ---- the E tiles start on their way at once: one barrier per tile, rows by the lanes of warp 0
  if (warp == 0) {
    const uint64_t pol = policy_evict_first();
    for (int ti = t_begin; ti < t_end; ++ti) {
      const ResTile tl = a.tiles[ti];
      if (tl.plain) continue;
      const LayerDev& L = t.layers[tl.layer];
      const float* E = L.E + ((size_t)tl.worker * L.n + tl.row0) * L.m + tl.col0;
      float* dst = resident + tl.smem_off;
      uint64_t* bar = sh.tile_bar + (ti - t_begin);
      if (lane == 0) mbar_arrive_expect_tx(bar, (uint32_t)tl.nrows * tl.ncols * 4u);
      __syncwarp();
      if (tl.ncols == L.m) {
        if (lane == 0) bulk_load_hint(dst, E, (uint32_t)tl.nrows * tl.ncols * 4u, bar, pol);
      } else {
        for (int row = lane; row < tl.nrows; row += 32)
          bulk_load_hint(dst + row * tl.ncols, E + (size_t)row * L.m, (uint32_t)tl.ncols * 4u, bar, pol);
      }
    }
  }
  if (tid == 0) {
    // the two counter sets alternate between launches; this launch clears the other one for the next
    const uint32_t seq = ld_acquire_u32(a.sync);
    sh.slot = seq & 1u;
    if (blockIdx.x == 0)
      for (int k = 0; k < kResBarriers; ++k) a.sync[1 + ((seq & 1u) ^ 1u) * kResBarriers + k] = 0u;
  }
  __syncthreads();

  bool ok = true;
  int nbar = 0, nstamp = 0;
  // timeline of the round as CTA 0 sees it (nanoseconds of the global timer): start, end of its pass 1, then
  // the moment it leaves each grid barrier, then the end; read back through lqsgd_round_timeline
  auto stamp = [&]() {
    if (blockIdx.x == 0 && tid == 0 && nstamp < kResStamps) a.stamps[nstamp] = global_ns();
    ++nstamp;
  };
  stamp();
  // Leaving early: the E copies of pass 1 may still be in flight towards this CTA's shared memory.
  auto leave = [&](int layer_for_status) {
    if (tid == 0) {
      report_timeout(t, layer_for_status);
      const uint32_t limit = wait_limit_of(sh.wait_ctl);
      for (int ti = t_begin; ti < t_end; ++ti)
        if (!a.tiles[ti].plain)
          for (uint32_t i = 0; i < limit && !mbar_try(sh.tile_bar + (ti - t_begin), 0); ++i) {}
      if (blockIdx.x == 0) atomicAdd(a.sync, 1u);
    }
  };

  // ---- A: pass 1
  float* red1 = reinterpret_cast<float*>(scratch);
  for (int ti = t_begin; ti < t_end && ok; ++ti) {
    const ResTile tl = a.tiles[ti];
    if (tl.plain) res_pass1_plain<RP>(t, tl, resident + tl.smem_off);
    else ok = res_pass1_tile<RP>(t, tl, resident + tl.smem_off, sh.tile_bar + (ti - t_begin), red1, sh);
    __syncthreads();
  }
  if (!ok) { leave(t_end > t_begin ? a.tiles[t_begin].layer : 0); return; }
  stamp();
  if (!grid_barrier(a, t, sh, nbar++)) { leave(0); return; }
  stamp();

  // ---- B: Orthonormalize (small layers whole, tall layers' Gram blocks), the 1-D tensors
  {
    const int total = a.nfbS + a.nfbP + a.vj.nchunks;
    for (int j = blockIdx.x; j < total; j += gridDim.x) {
      if (j < a.nfbS) step_orth_small<RP>(t, a.fbS[j], scratch);
      else if (j < a.nfbS + a.nfbP) step_reduce_gram<RP>(t, a.fbP[j - a.nfbS], scratch);
      else step_vectors(a.vj, j - a.nfbS - a.nfbP, t.payload, t.payload_stride, t.W);
      __syncthreads();
    }
  }
  if (!grid_barrier(a, t, sh, nbar++)) { leave(0); return; }
  stamp();
  if (a.nfbP > 0) {
    for (int j = blockIdx.x; j < a.nfbP; j += gridDim.x) {
      step_apply<RP>(t, a.fbP[j], scratch);
      __syncthreads();
    }
    if (!grid_barrier(a, t, sh, nbar++)) { leave(0); return; }
  stamp();
  }
  // ---- D: P_bar of the tiles' own rows, pass 2; then this CTA's share of the exchange of P proper
  {
    float* pb = reinterpret_cast<float*>(scratch);
    float* red = pb + kResMaxTileRows * RP;
    for (int ti = t_begin; ti < t_end; ++ti) {
      const ResTile tl = a.tiles[ti];
      exchange_rows_local<RP, kResThreads, true>(t, a.qp, 0, t.layers[tl.layer], tl.row0, tl.nrows, pb, tid, xl);
      res_pass2_tile<RP>(t, tl, resident + tl.smem_off, pb, red);
    }
  }
  if (!grid_barrier(a, t, sh, nbar++)) { leave(0); return; }
  stamp();
  // ---- E: Q_w (dealt from CTA 0 up); the exchange of P proper (payloads, P_bar for pass 3) from the last CTA
  // down: nothing before pass 3 waits for it, and this interval has CTAs to spare
  for (int j = blockIdx.x; j < a.nfbQ; j += gridDim.x) {
    step_q_reduce<RP>(t, a.fbQ[j], scratch);
    __syncthreads();
  }
  {
    for (int j = (int)(gridDim.x - 1 - blockIdx.x); j < a.nchP; j += gridDim.x) {
      step_exchange<RP>(t, a.qp, 0, a.chP[j], scratch);
      __syncthreads();
    }
  }
  if (!grid_barrier(a, t, sh, nbar++)) { leave(0); return; }
  stamp();
  // ---- G: Q_bar of the tiles' own columns, pass 3, tiles back to E by bulk store; then the exchange of Q proper
  {
    float* pb = reinterpret_cast<float*>(scratch);
    float* qb = pb + kResMaxTileRows * RP;
    const uint64_t pol = policy_evict_first();
    for (int ti = t_begin; ti < t_end; ++ti) {
      const ResTile tl = a.tiles[ti];
      exchange_rows_local<RP, kResThreads, true>(t, a.qq, 1, t.layers[tl.layer], tl.col0, tl.ncols, qb, tid, xl);
      res_pass3_tile<RP>(t, tl, resident + tl.smem_off, pb, qb);
      if (!tl.plain && warp == 0) {
        const LayerDev& L = t.layers[tl.layer];
        float* E = L.E + ((size_t)tl.worker * L.n + tl.row0) * L.m + tl.col0;
        const float* srcp = resident + tl.smem_off;
        if (tl.ncols == L.m) {
          if (lane == 0) bulk_store_hint(E, srcp, (uint32_t)tl.nrows * tl.ncols * 4u, pol);
        } else {
          for (int row = lane; row < tl.nrows; row += 32)
            bulk_store_hint(E + (size_t)row * L.m, srcp + row * tl.ncols, (uint32_t)tl.ncols * 4u, pol);
        }
        bulk_commit();
      }
    }
    for (int j = blockIdx.x; j < a.nchQ; j += gridDim.x) {
      step_exchange<RP>(t, a.qq, 1, a.chQ[j], scratch);
      __syncthreads();
    }
    if (warp == 0) bulk_wait_all0();
  }
  stamp();
  if (tid == 0 && blockIdx.x == 0) {
    a.stamps[kResStamps] = (uint64_t)nstamp;
    atomicAdd(a.sync, 1u);     // the next launch takes the other counter set
  }
}

}  // namespace

size_t resident_scratch_bytes(int RP) {
  switch (RP) {
    case 1: return ResScratch<1>::value + kResControlBytes;
    case 2: return ResScratch<2>::value + kResControlBytes;
    case 4: return ResScratch<4>::value + kResControlBytes;
    case 8: return ResScratch<8>::value + kResControlBytes;
    default: return 0;
  }
}

cudaError_t launch_resident(int RP, const Tables& t, const ResidentArgs& a, int grid, size_t smem_bytes, cudaStream_t stream) {
  auto go = [&](auto kernel) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kResThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;      // every CTA resident at once: what the grid barriers rely on
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, t, a);
  };
  switch (RP) {
    case 1: return go(resident_round_kernel<1>);
    case 2: return go(resident_round_kernel<2>);
    case 4: return go(resident_round_kernel<4>);
    case 8: return go(resident_round_kernel<8>);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t resident_max_grid(int RP, size_t smem_bytes, int sm_count, int* grid_out) {
  int occ = 0;
  cudaError_t e = cudaSuccess;
  auto q = [&](auto kernel) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kResThreads, smem_bytes);
  };
  switch (RP) {
    case 1: q(resident_round_kernel<1>); break;
    case 2: q(resident_round_kernel<2>); break;
    case 4: q(resident_round_kernel<4>); break;
    case 8: q(resident_round_kernel<8>); break;
    default: return cudaErrorInvalidValue;
  }
  *grid_out = occ > 0 ? sm_count : 0;
  return e;
}

}  // namespace lqsgd

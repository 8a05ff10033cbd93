// Bulk-copy (TMA) staged versions of the three streaming passes, used for every layer whose
// rows are 16-byte aligned (m % 4 == 0) and padded rank <= 8.
//
// One CTA per SM.  512 consumer threads compute; a loader warp brings 16-row x <=512-column
// slabs of G / E / M into a ring of shared-memory stages with cp.async.bulk (one 1-D bulk copy
// per row segment, completion counted on an mbarrier); a storer warp writes finished slabs
// (M in pass 1, E in pass 3) back with bulk stores.  The bytes in flight are set by the ring
// (up to ~190 KB per SM), not by registers, and the consumers touch global memory only for the
// small factor data.
//
// Consumer mapping (all passes): thread = (row group g of 4, column quad cv of 128): it owns
// 4 consecutive columns of the tile for 4 rows of every stage, so the rows of Q it needs
// (pass 1, pass 3) stay in registers for the whole tile.
//
// Every wait on an mbarrier is bounded: after kSpinLimit polls the waiter raises the CTA's abort
// flag and sets LQSGD_STATUS_TIMEOUT in the layer's status word; all roles then leave their
// loops (consumers at their next common barrier), the loader drains the copies it has in flight
// (bounded) and the kernel returns.
#include "lqsgd_dev.h"

#include <math.h>

namespace lqsgd {
namespace {

constexpr int kTileCols = kStreamTileCols;   // 512
constexpr int kStageRows = kStreamStageRows; // 16
constexpr int kGroups = 4;
constexpr int kColThreads = 128;
constexpr int kConsumers = kGroups * kColThreads;      // 512
constexpr int kConsumerWarps = kConsumers / 32;        // 16
constexpr int kThreads = kConsumers + 64;              // + loader warp + storer warp
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr uint32_t kStatusTimeout = 16u;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises *abort_flag) if the phase did not complete in time,
// or at once if another thread already raised the flag.
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_test(b, parity)) return true;
    if (*abort_flag) return false;
    if (i > 64) __nanosleep(40);
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }

// Same log-step reduction as in the register-path kernels: sums v[i] over the 32 lanes; afterwards
// lane l holds indices [l*N/32, (l+1)*N/32) (N >= 32) or index l / (32/N) (N < 32).
template <int N, int O>
__device__ __forceinline__ void warp_transpose_reduce(float* v, int lane) {
  if constexpr (O >= 1) {
    if constexpr (N > 1) {
      constexpr int H = N / 2;
      const bool up = (lane & O) != 0;
#pragma unroll
      for (int i = 0; i < H; ++i) {
        const float a = v[i], b = v[i + H];
        v[i] = (up ? b : a) + __shfl_xor_sync(0xffffffffu, up ? a : b, O);
      }
      warp_transpose_reduce<H, O / 2>(v, lane);
    } else {
      v[0] += __shfl_xor_sync(0xffffffffu, v[0], O);
      warp_transpose_reduce<1, O / 2>(v, lane);
    }
  }
}

template <int RP>
__device__ __forceinline__ void load_q_slice4(const float* __restrict__ Qt, int mt, int col, float (&q)[4 * RP]) {
#pragma unroll
  for (int j = 0; j < RP; ++j) {
    const float4 v = __ldg(reinterpret_cast<const float4*>(Qt + (size_t)j * mt + col));
    q[0 * RP + j] = v.x; q[1 * RP + j] = v.y; q[2 * RP + j] = v.z; q[3 * RP + j] = v.w;
  }
}

// Shared-memory ring common to the three passes.
struct Ring {
  uint64_t* full;      // [NST] loads landed (tx bytes)
  uint64_t* consumed;  // [NST] consumers done (one arrival per consumer warp)
  uint64_t* empty;     // [NST] stage may be refilled (storer, or consumers when nothing is stored)
  volatile int* abort_flag;
};

__device__ __forceinline__ void report_timeout(const Tables& t, int layer) { atomicOr(&t.status[layer], kStatusTimeout); }

// Loader drain on abort: the stages it has filled but nobody will consume still have copies in
// flight; poll their barriers (bounded) so that no copy targets the CTA's memory after exit.
template <int NST>
__device__ __forceinline__ void loader_drain(const Ring& r, uint32_t issued, uint32_t first_unfinished) {
  for (uint32_t it = first_unfinished; it < issued; ++it) {
    uint64_t* b = r.full + (it % NST);
    const uint32_t parity = (it / NST) & 1;
    for (uint32_t i = 0; i < kSpinLimit && !mbar_test(b, parity); ++i) __nanosleep(40);
  }
}

constexpr int kStageFloats = kStageRows * kTileCols;   // 8192 floats = 32 KB per slab

__device__ __forceinline__ void ring_init(const Ring& r, int nst, bool stores) {
  if (threadIdx.x == 0) {
    for (int s = 0; s < nst; ++s) {
      mbar_init(r.full + s, 1);                              // the loader's expect_tx arrival
      mbar_init(r.consumed + s, kConsumerWarps);
      mbar_init(r.empty + s, stores ? 1 : kConsumerWarps);   // storer, or the consumer warps directly
    }
    *r.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  __syncthreads();
}

// lane 0 waits, the warp learns the outcome
__device__ __forceinline__ bool warp_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag, int lane) {
  int ok = 1;
  if (lane == 0) ok = mbar_wait(b, parity, abort_flag) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// ---------------------------------------------------------------------------------------
// pass 1: M = G + E (Eq. 8) over E, partial P = M Q (Alg. 1).  Tile = up to 64 rows x 512 cols.
// ---------------------------------------------------------------------------------------
template <int RP, int NST>
__global__ void __launch_bounds__(kThreads, 1)
stream_pass1_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* sG = reinterpret_cast<float*>(smem_raw);
  float* sE = sG + NST * kStageFloats;
  float* red = sE + NST * kStageFloats;                       // [2][kGroups][4][4*RP]
  uint64_t* bars = reinterpret_cast<uint64_t*>(red + 2 * kGroups * 4 * 4 * RP);
  const Ring ring{bars, bars + NST, bars + 2 * NST, reinterpret_cast<volatile int*>(bars + 3 * NST)};
  ring_init(ring, NST, true);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint32_t it = 0;

  if (warp == kConsumerWarps) {                 // ---- loader
    bool ok = true;
    int last_layer = 0;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      const Tile tl = tiles[ti];
      const LayerDev& L = t.layers[tl.layer];
      last_layer = tl.layer;
      const int m = L.m;
      const float* G = t.grads[(size_t)tl.layer * t.W + tl.worker];
      const float* E = L.E + (size_t)tl.worker * L.n * m;
      const uint32_t rowbytes = (uint32_t)tl.ncols * 4u;
      for (int sr = 0; sr < tl.nrows; sr += kStageRows, ++it) {
        const int s = it % NST;
        const uint32_t k = it / NST;
        const int rows = min(kStageRows, tl.nrows - sr);
        if (k > 0) ok = warp_wait(ring.empty + s, (k - 1) & 1, ring.abort_flag, lane);
        if (!ok) break;
        if (lane == 0) mbar_arrive_expect_tx(ring.full + s, 2u * rows * rowbytes);
        __syncwarp();
        const int arr = lane >> 4, row = lane & 15;
        if (row < rows) {
          const size_t off = (size_t)(tl.row0 + sr + row) * m + tl.col0;
          bulk_load((arr ? sE : sG) + s * kStageFloats + row * kTileCols, (arr ? E : G) + off, rowbytes, ring.full + s);
        }
      }
    }
    if (!ok) {
      if (lane == 0) { report_timeout(t, last_layer); loader_drain<NST>(ring, it, it > (uint32_t)NST ? it - NST : 0); }
    }
    return;
  }
  if (warp == kConsumerWarps + 1) {             // ---- storer: M slabs back over E
    bool ok = true;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      const Tile tl = tiles[ti];
      const LayerDev& L = t.layers[tl.layer];
      float* E = L.E + (size_t)tl.worker * L.n * L.m;
      const uint32_t rowbytes = (uint32_t)tl.ncols * 4u;
      for (int sr = 0; sr < tl.nrows; sr += kStageRows, ++it) {
        const int s = it % NST;
        const int rows = min(kStageRows, tl.nrows - sr);
        ok = warp_wait(ring.consumed + s, (it / NST) & 1, ring.abort_flag, lane);
        if (!ok) break;
        if (lane < rows)
          bulk_store(E + (size_t)(tl.row0 + sr + lane) * L.m + tl.col0, sE + s * kStageFloats + lane * kTileCols, rowbytes);
        bulk_commit();
        bulk_wait_read0();
        __syncwarp();
        if (lane == 0) mbar_arrive(ring.empty + s);
      }
    }
    bulk_wait_all0();
    return;
  }

  // ---- consumers
  const int g = tid / kColThreads, cv = tid % kColThreads, wig = cv >> 5;
  constexpr int N = 4 * RP;
  int buf = 0;
  for (int ti = blockIdx.x; ti < ntiles; ti += gridDim.x) {
    const Tile tl = tiles[ti];
    const LayerDev& L = t.layers[tl.layer];
    const bool active = cv * 4 < tl.ncols;
    float q[4 * RP];
    if (active) load_q_slice4<RP>(L.Qt, L.mt, tl.col0 + cv * 4, q);
    else {
#pragma unroll
      for (int i = 0; i < 4 * RP; ++i) q[i] = 0.f;
    }
    float* Pp = L.Ppart + ((size_t)tl.worker * L.ncc + tl.part) * (size_t)L.n * RP;
    for (int sr = 0; sr < tl.nrows; sr += kStageRows, ++it) {
      const int s = it % NST;
      const int rows = min(kStageRows, tl.nrows - sr);
      const bool ok = mbar_wait(ring.full + s, (it / NST) & 1, ring.abort_flag);
      float acc[N];
#pragma unroll
      for (int i = 0; i < N; ++i) acc[i] = 0.f;
      if (ok && active) {
        const float4* pg = reinterpret_cast<const float4*>(sG + s * kStageFloats) + cv;
        float4* pe = reinterpret_cast<float4*>(sE + s * kStageFloats) + cv;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int lr = g * 4 + u;
          if (lr < rows) {
            const float4 gv = pg[lr * (kTileCols / 4)];
            const float4 ev = pe[lr * (kTileCols / 4)];
            const float4 mv = make_float4(gv.x + ev.x, gv.y + ev.y, gv.z + ev.z, gv.w + ev.w);
            pe[lr * (kTileCols / 4)] = mv;
#pragma unroll
            for (int j = 0; j < RP; ++j) {
              float a = acc[u * RP + j];
              a = fmaf(mv.x, q[0 * RP + j], a);
              a = fmaf(mv.y, q[1 * RP + j], a);
              a = fmaf(mv.z, q[2 * RP + j], a);
              a = fmaf(mv.w, q[3 * RP + j], a);
              acc[u * RP + j] = a;
            }
          }
        }
      }
      fence_async_smem();                       // M slab written by this thread -> visible to the bulk store
      __syncwarp();
      if (lane == 0) mbar_arrive(ring.consumed + s);
      warp_transpose_reduce<N, 16>(acc, lane);
      float* rd = red + ((buf * kGroups + g) * 4 + wig) * N;
      if constexpr (N >= 32) {
#pragma unroll
        for (int i = 0; i < N / 32; ++i) rd[lane * (N / 32) + i] = acc[i];
      } else {
        if ((lane % (32 / N)) == 0) rd[lane / (32 / N)] = acc[0];
      }
      consumer_barrier();
      if (*ring.abort_flag) {                   // uniform: raised before the barrier
        if (tid == 0) report_timeout(t, tl.layer);
        return;
      }
      if (tid < kStageRows * RP) {
        const int lr = tid / RP, j = tid % RP;
        if (lr < rows) {
          const float* r0 = red + ((buf * kGroups + (lr >> 2)) * 4) * N + (lr & 3) * RP + j;
          const float sum = ((r0[0] + r0[N]) + r0[2 * N]) + r0[3 * N];   // column quarters in order
          Pp[(size_t)(tl.row0 + sr + lr) * RP + j] = sum;
        }
      }
      buf ^= 1;
    }
  }
}

// ---------------------------------------------------------------------------------------
// pass 2: partial Q = M^T P_bar (Alg. 1).  Tile = a row chunk x 512 columns; a stage carries 16
// rows of M and the same 16 rows of P_bar.  A thread sums its 4 columns over its group's rows;
// the four row groups are then added in a fixed order through shared memory.
// ---------------------------------------------------------------------------------------
template <int RP, int NST>
__global__ void __launch_bounds__(kThreads, 1)
stream_pass2_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* sM = reinterpret_cast<float*>(smem_raw);
  float* sP = sM + NST * kStageFloats;                         // [NST][16*RP]
  float* red = sP + NST * kStageRows * RP;                     // [2][4*RP][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(red + 2 * 4 * RP * kColThreads);
  const Ring ring{bars, bars + NST, bars + 2 * NST, reinterpret_cast<volatile int*>(bars + 3 * NST)};
  ring_init(ring, NST, false);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint32_t it = 0;

  if (warp == kConsumerWarps) {                 // ---- loader
    bool ok = true;
    int last_layer = 0;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      const Tile tl = tiles[ti];
      const LayerDev& L = t.layers[tl.layer];
      last_layer = tl.layer;
      const int m = L.m;
      const float* M = L.E + (size_t)tl.worker * L.n * m;
      const uint32_t rowbytes = (uint32_t)tl.ncols * 4u;
      for (int sr = 0; sr < tl.nrows; sr += kStageRows, ++it) {
        const int s = it % NST;
        const uint32_t k = it / NST;
        const int rows = min(kStageRows, tl.nrows - sr);
        if (k > 0) ok = warp_wait(ring.empty + s, (k - 1) & 1, ring.abort_flag, lane);
        if (!ok) break;
        const uint32_t pbytes = (uint32_t)kStageRows * RP * 4u;     // P_bar is padded to whole 16-row blocks
        if (lane == 0) mbar_arrive_expect_tx(ring.full + s, rows * rowbytes + pbytes);
        __syncwarp();
        if (lane < rows)
          bulk_load(sM + s * kStageFloats + lane * kTileCols, M + (size_t)(tl.row0 + sr + lane) * m + tl.col0, rowbytes,
                    ring.full + s);
        if (lane == 16)
          bulk_load(sP + s * kStageRows * RP, L.Pbar + (size_t)(tl.row0 + sr) * RP, pbytes, ring.full + s);
      }
    }
    if (!ok && lane == 0) { report_timeout(t, last_layer); loader_drain<NST>(ring, it, it > (uint32_t)NST ? it - NST : 0); }
    return;
  }
  if (warp > kConsumerWarps) return;            // no storer in this pass

  const int g = tid / kColThreads, cv = tid % kColThreads;
  constexpr int N = 4 * RP;
  for (int ti = blockIdx.x; ti < ntiles; ti += gridDim.x) {
    const Tile tl = tiles[ti];
    const LayerDev& L = t.layers[tl.layer];
    const bool active = cv * 4 < tl.ncols;
    float acc[N];                                // acc[k * RP + j]: column k of the quad, rank j
#pragma unroll
    for (int i = 0; i < N; ++i) acc[i] = 0.f;
    for (int sr = 0; sr < tl.nrows; sr += kStageRows, ++it) {
      const int s = it % NST;
      const int rows = min(kStageRows, tl.nrows - sr);
      const bool ok = mbar_wait(ring.full + s, (it / NST) & 1, ring.abort_flag);
      if (ok && active) {
        const float4* pm = reinterpret_cast<const float4*>(sM + s * kStageFloats) + cv;
        const float* pp = sP + s * kStageRows * RP;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int lr = g * 4 + u;
          if (lr < rows) {
            const float4 mv = pm[lr * (kTileCols / 4)];
            float p[RP];
#pragma unroll
            for (int j = 0; j < RP; ++j) p[j] = pp[lr * RP + j];
#pragma unroll
            for (int j = 0; j < RP; ++j) {
              acc[0 * RP + j] = fmaf(mv.x, p[j], acc[0 * RP + j]);
              acc[1 * RP + j] = fmaf(mv.y, p[j], acc[1 * RP + j]);
              acc[2 * RP + j] = fmaf(mv.z, p[j], acc[2 * RP + j]);
              acc[3 * RP + j] = fmaf(mv.w, p[j], acc[3 * RP + j]);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(ring.empty + s);
    }
    // (g0 + g2) + (g1 + g3): groups 2 and 3 hand over first, then group 1
    float* regA = red;
    float* regB = red + N * kColThreads;
    if (g >= 2) {
      float* dst = (g == 2) ? regA : regB;
#pragma unroll
      for (int k = 0; k < N; ++k) dst[k * kColThreads + cv] = acc[k];
    }
    consumer_barrier();
    if (*ring.abort_flag) {
      if (tid == 0) report_timeout(t, tl.layer);
      return;
    }
    if (g < 2) {
      const float* src = (g == 0) ? regA : regB;
#pragma unroll
      for (int k = 0; k < N; ++k) acc[k] += src[k * kColThreads + cv];
    }
    consumer_barrier();
    if (g == 1) {
#pragma unroll
      for (int k = 0; k < N; ++k) regA[k * kColThreads + cv] = acc[k];
    }
    consumer_barrier();
    if (g == 0 && active) {
#pragma unroll
      for (int k = 0; k < N; ++k) acc[k] += regA[k * kColThreads + cv];
      float* dst = L.Qpart + (((size_t)tl.worker * L.nrb + tl.part) * (size_t)L.m + tl.col0 + cv * 4) * RP;
      if constexpr (N % 4 == 0) {
#pragma unroll
        for (int i = 0; i < N / 4; ++i)
          reinterpret_cast<float4*>(dst)[i] = make_float4(acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3]);
      } else {
#pragma unroll
        for (int i = 0; i < N; ++i) dst[i] = acc[i];
      }
    }
    consumer_barrier();                          // regA is free again before the next tile ends
  }
}

// ---------------------------------------------------------------------------------------
// pass 3: G_hat = P_bar Q_bar^T (Eq. 6), E_w = M_w - G_hat (Eq. 7).  Tile = rows x 512 columns,
// all workers: for every 16-row block the workers' M slabs follow one another through the ring;
// G_hat of the block is formed once (with the first worker's slab) and kept in registers.
// ---------------------------------------------------------------------------------------
template <int RP, int NST>
__global__ void __launch_bounds__(kThreads, 1)
stream_pass3_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  float* sM = reinterpret_cast<float*>(smem_raw);
  float* sP = sM + NST * kStageFloats;                         // [NST][16*RP]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sP + NST * kStageRows * RP);
  const Ring ring{bars, bars + NST, bars + 2 * NST, reinterpret_cast<volatile int*>(bars + 3 * NST)};
  ring_init(ring, NST, true);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int W = t.W;
  uint32_t it = 0;

  if (warp == kConsumerWarps) {                 // ---- loader
    bool ok = true;
    int last_layer = 0;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      const Tile tl = tiles[ti];
      const LayerDev& L = t.layers[tl.layer];
      last_layer = tl.layer;
      const int m = L.m;
      const size_t plane = (size_t)L.n * m;
      const uint32_t rowbytes = (uint32_t)tl.ncols * 4u;
      const uint32_t pbytes = (uint32_t)kStageRows * RP * 4u;
      for (int sr = 0; sr < tl.nrows && ok; sr += kStageRows) {
        const int rows = min(kStageRows, tl.nrows - sr);
        for (int w = 0; w < W; ++w, ++it) {
          const int s = it % NST;
          const uint32_t k = it / NST;
          if (k > 0) ok = warp_wait(ring.empty + s, (k - 1) & 1, ring.abort_flag, lane);
          if (!ok) break;
          if (lane == 0) mbar_arrive_expect_tx(ring.full + s, rows * rowbytes + (w == 0 ? pbytes : 0u));
          __syncwarp();
          if (lane < rows)
            bulk_load(sM + s * kStageFloats + lane * kTileCols,
                      L.E + (size_t)w * plane + (size_t)(tl.row0 + sr + lane) * m + tl.col0, rowbytes, ring.full + s);
          if (lane == 16 && w == 0)
            bulk_load(sP + s * kStageRows * RP, L.Pbar + (size_t)(tl.row0 + sr) * RP, pbytes, ring.full + s);
        }
      }
    }
    if (!ok && lane == 0) { report_timeout(t, last_layer); loader_drain<NST>(ring, it, it > (uint32_t)NST ? it - NST : 0); }
    return;
  }
  if (warp == kConsumerWarps + 1) {             // ---- storer: E slabs
    bool ok = true;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      const Tile tl = tiles[ti];
      const LayerDev& L = t.layers[tl.layer];
      const size_t plane = (size_t)L.n * L.m;
      const uint32_t rowbytes = (uint32_t)tl.ncols * 4u;
      for (int sr = 0; sr < tl.nrows && ok; sr += kStageRows) {
        const int rows = min(kStageRows, tl.nrows - sr);
        for (int w = 0; w < W; ++w, ++it) {
          const int s = it % NST;
          ok = warp_wait(ring.consumed + s, (it / NST) & 1, ring.abort_flag, lane);
          if (!ok) break;
          if (lane < rows)
            bulk_store(L.E + (size_t)w * plane + (size_t)(tl.row0 + sr + lane) * L.m + tl.col0,
                       sM + s * kStageFloats + lane * kTileCols, rowbytes);
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

  const int g = tid / kColThreads, cv = tid % kColThreads;
  for (int ti = blockIdx.x; ti < ntiles; ti += gridDim.x) {
    const Tile tl = tiles[ti];
    const LayerDev& L = t.layers[tl.layer];
    const bool active = cv * 4 < tl.ncols;
    const int col = tl.col0 + cv * 4;
    float q[4 * RP];
    if (active) load_q_slice4<RP>(L.Qt, L.mt, col, q);
    float* Gh = t.ghat[tl.layer];
    for (int sr = 0; sr < tl.nrows; sr += kStageRows) {
      const int rows = min(kStageRows, tl.nrows - sr);
      float4 gh[4];
      for (int w = 0; w < W; ++w, ++it) {
        const int s = it % NST;
        const bool ok = mbar_wait(ring.full + s, (it / NST) & 1, ring.abort_flag);
        if (ok && active) {
          float4* pm = reinterpret_cast<float4*>(sM + s * kStageFloats) + cv;
          if (w == 0) {
            const float* pp = sP + s * kStageRows * RP;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int lr = g * 4 + u;
              if (lr < rows) {
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                for (int j = 0; j < RP; ++j) {
                  const float p = pp[lr * RP + j];
                  a0 = fmaf(p, q[0 * RP + j], a0);
                  a1 = fmaf(p, q[1 * RP + j], a1);
                  a2 = fmaf(p, q[2 * RP + j], a2);
                  a3 = fmaf(p, q[3 * RP + j], a3);
                }
                gh[u] = make_float4(a0, a1, a2, a3);
                __stcs(reinterpret_cast<float4*>(Gh + (size_t)(tl.row0 + sr + lr) * L.m + col), gh[u]);
              }
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int lr = g * 4 + u;
            if (lr < rows) {
              const float4 mv = pm[lr * (kTileCols / 4)];
              pm[lr * (kTileCols / 4)] = make_float4(mv.x - gh[u].x, mv.y - gh[u].y, mv.z - gh[u].z, mv.w - gh[u].w);
            }
          }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(ring.consumed + s);
      }
    }
    if (*ring.abort_flag) {                      // not a barrier: each consumer leaves on its own
      if (tid == 0) report_timeout(t, tl.layer);
      return;
    }
  }
}

size_t smem_pass1(int RP, int NST) { return (size_t)NST * 2 * kStageFloats * 4 + 2 * kGroups * 4 * 4 * RP * 4 + (3 * NST + 1) * 8; }
size_t smem_pass2(int RP, int NST) {
  return (size_t)NST * (kStageFloats + kStageRows * RP) * 4 + 2 * 4 * RP * kColThreads * 4 + (3 * NST + 1) * 8;
}
size_t smem_pass3(int RP, int NST) { return (size_t)NST * (kStageFloats + kStageRows * RP) * 4 + (3 * NST + 1) * 8; }

template <typename K>
cudaError_t launch_staged(K kernel, size_t smem, const Tables& t, const Tile* tiles, int ntiles, Launch l) {
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kernel<<<l.grid, kThreads, smem, l.stream>>>(t, tiles, ntiles);
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

constexpr int kNst1 = 3, kNst2 = 5, kNst3 = 6;

cudaError_t launch_stream_pass1(int rp, const Tables& t, const Tile* tiles, int ntiles, Launch l) {
  if (ntiles == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP8(rp, return launch_staged(stream_pass1_kernel<RP, kNst1>, smem_pass1(RP, kNst1), t, tiles, ntiles, l));
  return cudaSuccess;
}
cudaError_t launch_stream_pass2(int rp, const Tables& t, const Tile* tiles, int ntiles, Launch l) {
  if (ntiles == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP8(rp, return launch_staged(stream_pass2_kernel<RP, kNst2>, smem_pass2(RP, kNst2), t, tiles, ntiles, l));
  return cudaSuccess;
}
cudaError_t launch_stream_pass3(int rp, const Tables& t, const Tile* tiles, int ntiles, Launch l) {
  if (ntiles == 0) return cudaSuccess;
  LQSGD_DISPATCH_RP8(rp, return launch_staged(stream_pass3_kernel<RP, kNst3>, smem_pass3(RP, kNst3), t, tiles, ntiles, l));
  return cudaSuccess;
}

}  // namespace lqsgd

// Helpers of the bulk-copy (TMA) staged passes in lqsgd_stream.cu, which serve every layer whose
// rows are 16-byte aligned (m % 4 == 0) and padded rank <= 8.
//
// One CTA per SM.  512 consumer threads compute; a loader warp brings slabs of G / E / M (a few
// rows of a wide tile, up to 36 KB) into a ring of shared-memory stages with cp.async.bulk,
// completion counted on an mbarrier; a storer warp writes finished slabs (M in pass 1, E in
// pass 3) back with bulk stores.  The bytes in flight are set by the ring, not by registers.
// The copy engine tracks a limited number of bulk copies, whatever their size, so a stage is
// made of few large copies: one per row segment of a tile up to 2048-6144 columns wide, and a
// single copy when the tile spans whole rows (then the rows are contiguous in memory).
//
// Consumer mapping (all passes): a thread owns 1-3 column quads (4 consecutive columns each) of
// the tile, for up to 4 or 8 rows of every stage; narrow tiles put several row groups side by
// side.  The rows of Q a thread needs (pass 1, pass 3) stay in registers for the whole tile.
//
// Every wait on an mbarrier is bounded: after kWaitLimit timed try_wait calls the waiter raises
// the CTA's abort flag; all roles then leave their loops (consumers at their next common
// barrier, where the layer's status word gets LQSGD_STATUS_TIMEOUT), the loader drains the
// copies it has in flight (bounded) and the kernel returns.
#pragma once
#include "lqsgd_dev.h"

#include <math.h>

namespace lqsgd {
namespace {

constexpr int kConsumers = kStreamConsumers;           // 512
constexpr int kConsumerWarps = kConsumers / 32;        // 16
constexpr int kThreads = kConsumers + 64;              // + loader warp + storer warp
constexpr int kSlab = kStreamSlabFloats;               // floats per stage per array
constexpr uint32_t kWaitLimit = 1u << 18;              // try_wait calls of <= ~1 us each (the default limit)
// The CTA's wait control lives in shared memory as consecutive ints: [0] the abort flag, [1] the limit of timed
// polls per wait (kWaitLimit unless a test shortened it); the functions below take the address of [0].
__device__ __forceinline__ void wait_ctl_init(volatile int* abort_flag, uint32_t limit_or_zero) {
  abort_flag[0] = 0;
  abort_flag[1] = (int)(limit_or_zero ? limit_or_zero : kWaitLimit);
}
__device__ __forceinline__ uint32_t wait_limit_of(volatile int* abort_flag) { return (uint32_t)abort_flag[1]; }
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
// One timed wait: the hardware suspends the thread until the phase completes or about a
// microsecond has passed (no spinning on the barrier word, which would compete with the copy
// engine's completion updates).
__device__ __forceinline__ bool mbar_try(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(b)), "r"(parity), "r"(1000u) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises the abort flag) if the phase did not complete in
// time, or as soon as another thread has raised the flag.
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
  const uint32_t limit = wait_limit_of(abort_flag);
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try(b, parity)) return true;
    if (*abort_flag) return false;
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
// L2 eviction policies for the streams: data that will not be read again in this round goes
// out first; data the next pass starts on (it walks the previous pass's order backwards) stays.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void bulk_load_hint(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(pol) : "memory");
}
__device__ __forceinline__ void bulk_store_hint(void* gdst, const void* smem_src, uint32_t bytes, uint64_t pol) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
               ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes), "l"(pol) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }

struct Ring {
  uint64_t* full;      // [NST] loads landed (tx bytes)
  uint64_t* consumed;  // [NST] consumers done (one arrival per consumer warp)
  uint64_t* empty;     // [NST] stage may be refilled (storer, or consumers when nothing is stored)
  volatile int* abort_flag;
};

__device__ __forceinline__ void ring_init(const Ring& r, int nst, bool stores, uint32_t wait_limit) {
  if (threadIdx.x == 0) {
    for (int s = 0; s < nst; ++s) {
      mbar_init(r.full + s, 1);                              // the loader's expect_tx arrival
      mbar_init(r.consumed + s, kConsumerWarps);
      mbar_init(r.empty + s, stores ? 1 : kConsumerWarps);   // storer, or the consumer warps directly
    }
    wait_ctl_init(r.abort_flag, wait_limit);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  __syncthreads();
}

// lane 0 waits, the warp learns the outcome (loader and storer warps)
__device__ __forceinline__ bool warp_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag, int lane) {
  int ok = 1;
  if (lane == 0) ok = mbar_wait(b, parity, abort_flag) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__device__ __forceinline__ void report_timeout(const Tables& t, int layer) { atomicOr(&t.status[layer], kStatusTimeout); }

// Loader drain on abort: stages it has filled but nobody will consume may still have copies in
// flight; wait (bounded) for them so that no copy targets the CTA's memory after it exits.
template <int NST>
__device__ __forceinline__ void loader_drain(const Ring& r, uint32_t issued) {
  const uint32_t limit = wait_limit_of(r.abort_flag);
  for (uint32_t it = issued > (uint32_t)NST ? issued - NST : 0; it < issued; ++it)
    for (uint32_t i = 0; i < limit && !mbar_try(r.full + (it % NST), (it / NST) & 1); ++i) {}
}

// What every role needs to know about a tile, read once from the tables.
struct TileCtx {
  int layer, worker, row0, nrows, col0, ncols, part;
  int m, n;
  bool contig;          // the tile spans whole rows: its rows are contiguous in memory
  StreamGeo geo;
};
template <int RP>
__device__ __forceinline__ TileCtx tile_ctx(const Tables& t, const Tile& tl) {
  TileCtx c;
  c.layer = tl.layer; c.worker = tl.worker; c.row0 = tl.row0; c.nrows = tl.nrows;
  c.col0 = tl.col0; c.ncols = tl.ncols; c.part = tl.part;
  c.m = t.layers[tl.layer].m; c.n = t.layers[tl.layer].n;
  c.contig = (tl.ncols == c.m);
  c.geo = stream_geo(tl.ncols, RP);
  return c;
}

// Loads `rows` row segments of the tile (starting at tile row sr) into a slab: one copy if the
// rows are contiguous, else one per row (lanes take rows).  Returns nothing; all on `bar`.
__device__ __forceinline__ void load_slab(float* slab, const float* src_tile, const TileCtx& c, int sr, int rows,
                                          uint64_t* bar, int lane, uint64_t pol) {
  if (c.contig) {
    if (lane == 0) bulk_load_hint(slab, src_tile + (size_t)sr * c.m, (uint32_t)rows * c.ncols * 4u, bar, pol);
  } else {
    for (int row = lane; row < rows; row += 32)
      bulk_load_hint(slab + row * c.ncols, src_tile + (size_t)(sr + row) * c.m, (uint32_t)c.ncols * 4u, bar, pol);
  }
}
__device__ __forceinline__ void store_slab(float* dst_tile, const float* slab, const TileCtx& c, int sr, int rows, int lane,
                                           uint64_t pol) {
  if (c.contig) {
    if (lane == 0) bulk_store_hint(dst_tile + (size_t)sr * c.m, slab, (uint32_t)rows * c.ncols * 4u, pol);
  } else {
    for (int row = lane; row < rows; row += 32)
      bulk_store_hint(dst_tile + (size_t)(sr + row) * c.m, slab + row * c.ncols, (uint32_t)c.ncols * 4u, pol);
  }
}

// Which quads and rows a consumer thread owns in a tile.
struct Owner {
  int g;          // row group (rows g, g + ng, ...)
  int cq;         // first quad; further quads are cq + 512, cq + 1024
  bool in_group;  // false for the few threads left over when 512 is not a multiple of tpr
};
__device__ __forceinline__ Owner owner_of(const StreamGeo& geo, int tid) {
  Owner o;
  o.g = tid / geo.tpr;
  o.cq = tid - o.g * geo.tpr;
  o.in_group = o.g < geo.ng;
  return o;
}

// q[(k * 4 + c) * RP + j] = Q[col0 + 4 * (cq + 512 k) + c][j], read from the transposed copy Qt
template <int RP, int QPT>
__device__ __forceinline__ void load_q(const float* __restrict__ Qt, int mt, int col0, const StreamGeo& geo,
                                       const Owner& o, float (&q)[QPT * 4 * RP]) {
#pragma unroll
  for (int k = 0; k < QPT; ++k) {
    const int quad = o.cq + k * kConsumers;
    const bool on = o.in_group && quad < geo.quads;
#pragma unroll
    for (int j = 0; j < RP; ++j) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (on) v = __ldg(reinterpret_cast<const float4*>(Qt + (size_t)j * mt + col0 + quad * 4));
      q[(k * 4 + 0) * RP + j] = v.x; q[(k * 4 + 1) * RP + j] = v.y;
      q[(k * 4 + 2) * RP + j] = v.z; q[(k * 4 + 3) * RP + j] = v.w;
    }
  }
}

// Uniform abort decision for the consumers: thread 0 samples the flag, a consumer barrier
// publishes the sample, everybody acts on the same value (the loader or storer may raise the
// flag at any moment, so reading it individually after a barrier could split the CTA).
// slot alternates 0 / 1 between consecutive calls.
__device__ __forceinline__ bool consumers_agree_abort(const Ring& r, volatile int* verdict, int slot, int tid) {
  if (tid == 0) verdict[slot] = *r.abort_flag;
  consumer_barrier();
  return verdict[slot] != 0;
}

}  // namespace
}  // namespace lqsgd

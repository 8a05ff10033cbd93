// Tensor-core passes of the LQ-SGD round for padded rank >= 16 (Blackwell, sm_100a).
//
// At rank 16 and above the products of Algorithm 1 cost more FP32 instructions per byte than the
// CUDA cores can issue at HBM speed.  These kernels run them on tcgen05, with fp32 accumulators
// in tensor memory (TMEM) and every fp32 operand fed as a sum of narrow terms.
//
// Pass 2 (Q_w = M_w^T P_bar, Alg. 1).  What a tcgen05.mma with M = 128 costs hardly depends on N <= 128
// (timing the first versions of this kernel: the feed of the A operand bounds it), so the streamed matrix must
// pass through the tensor core once, with as few instructions per byte as possible:
//   * M (the A operand, 128 columns of one worker's M per tile, lane = column) is split into two
//     bf16 terms, a = a1 + a2 (a1 the truncation of a to 8 mantissa bits, a2 = rn(a - a1): 16
//     significant bits, |a - a1 - a2| <= 2^-17 |a|), stored as a bf16 pair in ONE 32-bit TMEM
//     column, i.e. as two consecutive K elements;
//   * P_bar (the B operand) is split into three bf16 terms b = b1 + b2 + b3 (24 bits) that are
//     stacked along N (3 RP rows), each value repeated for the two K slots of its row.
// One kind::f16 MMA (K = 16) then covers 8 rows of M:  D[:, t RP + j] += sum_i (a1 + a2)_i b_t,ij
// and the epilogue adds the three N blocks.  Products are exact in the fp32 accumulator; the
// result differs from the fp32 product by the 2^-17 relative rounding of M only.
//
// Per CTA (one per SM, walking a list of tiles): a loader thread brings 32-row x 128-column
// pieces of M into a shared-memory ring with TMA tensor copies; three consumer warpgroups read
// them column-wise, split them and write the pairs to TMEM with tcgen05.st; a second loader
// brings the matching 32 rows of the stacked P_bar terms (kept transposed in global memory) as
// one 128-byte-swizzled K-major tile; one thread issues the MMAs; an epilogue warpgroup drains
// the accumulator (double-buffered) and stores Q_w.
//
// Every wait is bounded (see lqsgd_stream_common.cuh); on expiry the CTA raises its abort flag,
// all roles leave their loops, the loaders wait (bounded) for copies in flight, the MMA thread
// for its last commit, TMEM is released and the layer's status word gets LQSGD_STATUS_TIMEOUT.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstring>

#include "../../include/lqsgd.h"
#include "lqsgd_stream_common.cuh"

namespace lqsgd {
namespace {

constexpr int kTcThreads = 640;       // 20 warps: M loader, B loader, MMA, spare, 4 epilogue, 12 consumers
constexpr int kTcK = 32;              // rows of M per stage
constexpr int kTcCols = 128;          // columns of M per tile: the M extent of one MMA
constexpr int kTcPair = 2;            // stages per operand slot: the MMA thread waits, issues and commits once per
                                      // slot (a lone thread runs a few cycles per instruction: its bookkeeping counts)
constexpr int kTcAB = 4;              // ring of operand slots: A in TMEM, B in shared memory; deep enough to hide the
                                      // latency of the B copy, which can only start when its slot's MMAs are done
constexpr int kTcSlotK = kTcPair * kTcK;
constexpr int kTcGroups = 3;          // consumer warpgroups
constexpr uint32_t kTcMBytes = kTcK * kTcCols * 4;

__device__ __forceinline__ void tma_load_3d(void* smem_dst, const void* tmap, int x, int y, int z, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
               ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const void* tmap, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem_d] (+)= A[tmem_a] * B[desc]^T, bf16 inputs, fp32 accumulate; A from tensor memory.
__device__ __forceinline__ void tc_mma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
               ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row groups
// 1024 bytes apart; `addr` is the byte address of the first row plus the k-step offset.
__device__ __forceinline__ uint64_t tc_desc_sw128(uint32_t addr) {
  uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;              // leading byte offset: unused inside one swizzle atom
  d |= (uint64_t)(1024 >> 4) << 32;    // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;              // descriptor version of this architecture
  d |= (uint64_t)2 << 61;              // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t tc_idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
        "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
        "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Bounded wait of a single thread (the MMA issuer): a plain try first, which costs a few cycles
// when the phase is already complete, then the timed waits.
__device__ __forceinline__ bool thread_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
  uint32_t ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
  return ok ? true : mbar_wait(b, parity, abort_flag);
}
// Bounded wait for a loader's copies that nobody will consume (abort path).
__device__ __forceinline__ void drain(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  const uint32_t limit = wait_limit_of(abort_flag);
  for (uint32_t i = 0; i < limit && !mbar_try(bar, parity); ++i) {}
}

// ---------------------------------------------------------------------------------------
// Tiles handed out at run time (passes 1 and 3).  The SMs do not stream equally fast (two dies, memory partitions
// nearer or farther: 15 % between the quickest and the slowest in these passes), so equal shares dealt in
// advance leave the quick ones idle at the end.  CTA b starts on tile b; after that the loader thread draws the
// next index from a counter in global memory (asked for one tile ahead, so that the answer is there when it is
// needed) and announces it to the CTA's other roles through a small queue in shared memory.  Which CTA takes a
// tile does not change a result: every tile writes its own places.  The last CTA to leave puts the counter back
// to zero, so the next launch (or replay of a captured graph) finds it ready.
// ---------------------------------------------------------------------------------------
constexpr int kTqDepth = 4;
constexpr int kTqEnd = -1, kTqAbort = -2;
struct TileQueue {
  uint64_t* full;        // [kTqDepth] entry announced
  uint64_t* empty;       // [kTqDepth] every reader has taken the entry
  volatile int* idx;     // [kTqDepth] tile index, or kTqEnd
};
// the loader thread announces entry number seq
__device__ __forceinline__ bool tq_put(const TileQueue& q, uint32_t seq, int tile, volatile int* abort_flag) {
  const int s = seq % kTqDepth;
  if (!mbar_wait(q.empty + s, ((seq / kTqDepth) & 1) ^ 1, abort_flag)) return false;
  q.idx[s] = tile;
  mbar_arrive(q.full + s);
  return true;
}
// a reader thread takes entry number seq: the tile index, kTqEnd, or kTqAbort when a wait gave up
__device__ __forceinline__ int tq_take(const TileQueue& q, uint32_t seq, volatile int* abort_flag) {
  const int s = seq % kTqDepth;
  if (!mbar_wait(q.full + s, (seq / kTqDepth) & 1, abort_flag)) return kTqAbort;
  const int v = q.idx[s];
  mbar_arrive(q.empty + s);
  return v;
}
// a reader warp: lane 0 takes the entry, the warp learns it
__device__ __forceinline__ int tq_take_warp(const TileQueue& q, uint32_t seq, volatile int* abort_flag, int lane) {
  int v = 0;
  if (lane == 0) v = tq_take(q, seq, abort_flag);
  return __shfl_sync(0xffffffffu, v, 0);
}
// the loader thread's draw: the tiles after the fixed ones (fixed_per_cta per CTA), in the order asked for
__device__ __forceinline__ int tq_draw(int* sched, int ntiles, int fixed_per_cta = 1) {
  const int v = fixed_per_cta * (int)gridDim.x + atomicAdd(sched, 1);
  return v < ntiles ? v : kTqEnd;
}
// at the very end of the kernel, one thread per CTA: the last CTA to leave readies the counter for the next launch
__device__ __forceinline__ void tq_leave(int* sched) {
  __threadfence();
  if (atomicAdd(sched + 1, 1) == (int)gridDim.x - 1) {
    sched[0] = 0;
    sched[1] = 0;
    __threadfence();
  }
}

// Stages a tile takes: its rows in pieces of 32, rounded up to whole operand slots (a piece past
// the layer's last row reads as zeros and costs no memory traffic).
__device__ __forceinline__ int tile_stages(int nrows) {
  return (nrows + kTcSlotK - 1) / kTcSlotK * kTcPair;
}

template <int RP>
struct Pass2Cfg {
  static constexpr int kN = 3 * RP;                                      // stacked bf16 terms of P_bar
  static constexpr int kAB = RP <= 32 ? kTcAB : 2;                       // operand slots: at padded rank 64 a B stage is 24 KB
  static constexpr int kDStride = kN <= 64 ? 64 : (kN <= 128 ? 128 : 256);   // TMEM columns per accumulator
  static constexpr int kDBufs = (2 * kDStride + kAB * kTcSlotK <= 512) ? 2 : 1;
  static constexpr int kACol0 = kDBufs * kDStride;
  static constexpr int kTmemCols = (kACol0 + kAB * kTcSlotK) <= 256 ? 256 : 512;
  static constexpr uint32_t kBBytes = kN * 128;                          // one B stage: 3 RP rows of 64 bf16
  static constexpr uint32_t kBStride = (kBBytes + 1023) / 1024 * 1024;   // stages stay 1024-byte aligned
  static constexpr int kMStages = RP <= 16 ? 8 : 6;                      // ring of M pieces (16 KB each): what fits beside B
  static constexpr uint32_t kBOff = kMStages * kTcMBytes;
  static constexpr uint32_t kBarOff = kBOff + kAB * kTcPair * kBStride;
  static constexpr int kBars = 2 * kMStages + 2 * kAB + 2 + 2 + 1;
  static constexpr uint32_t kTotal = kBarOff + kBars * 8 + 16 + 1024;    // + abort flag, TMEM slot, alignment slack
  static_assert(kACol0 + kAB * kTcSlotK <= 512, "tensor memory");
  static_assert(kTotal <= 227 * 1024, "shared memory");
  // A ring's barrier tells its phases apart by parity alone: a waiter two phases ahead of the barrier would take
  // the phase before the one in progress for its own.  A consumer group can run at most the M ring (kMStages
  // pieces) ahead of the slowest group, and the MMA thread waits for all groups: that must stay below two turns of
  // the operand ring (2 kAB slots of kTcPair pieces).
  static_assert(kMStages < 2 * kAB * kTcPair, "a consumer must not get two turns of the operand ring ahead");
  static_assert(kN % 16 == 0 && kN <= 256, "N of one MMA");
};

template <int RP>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_pass2_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles, const uint8_t* __restrict__ maps) {
  pdl_wait();
  using S = Pass2Cfg<RP>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  float* mring = reinterpret_cast<float*>(base);
  uint8_t* bring = base + S::kBOff;
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + S::kBarOff);
  uint64_t* m_full = bars;                       // [S::kMStages] TMA landed
  uint64_t* m_empty = m_full + S::kMStages;       // [S::kMStages] consumer warps have the piece in registers
  uint64_t* ab_full = m_empty + S::kMStages;      // [S::kAB] slot ready: A written to TMEM (4 warps per stage) and B landed
  uint64_t* ab_empty = ab_full + S::kAB;          // [S::kAB] the MMAs that read buffer i have completed
  uint64_t* d_full = ab_empty + S::kAB;           // [2] accumulator complete
  uint64_t* d_empty = d_full + 2;                // [2] accumulator drained
  uint64_t* fin = d_empty + 2;                   // [1] every MMA of this CTA has completed
  volatile int* abort_flag = reinterpret_cast<volatile int*>(fin + 1);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(fin + 1) + 2;   // after the abort flag and the wait limit

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < S::kMStages; ++s) { mbar_init(m_full + s, 1); mbar_init(m_empty + s, 4); }
    for (int s = 0; s < S::kAB; ++s) { mbar_init(ab_full + s, 4 * kTcPair + 1); mbar_init(ab_empty + s, 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(d_full + s, 1); mbar_init(d_empty + s, 4); }
    mbar_init(fin, 1);
    wait_ctl_init(abort_flag, t.wait_limit);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)S::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ---- M loader
    uint32_t kc = 0;
    bool ok = true;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      const Tile tl = tiles[ti];
      const uint8_t* map = maps + (size_t)tl.layer * kTcMapsPerLayer * kTcMapBytes;
      const int nk = tile_stages(tl.nrows);
      for (int k = 0; k < nk; ++k, ++kc) {
        const int s = kc % S::kMStages;
        if (!warp_wait(m_empty + s, ((kc / S::kMStages) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        if (test_skips_stage(t, 2, kc)) continue;     // test support: this piece is not fetched, its waiters give up
        if (lane == 0) {
          mbar_arrive_expect_tx(m_full + s, kTcMBytes);
          tma_load_3d(mring + (size_t)s * (kTcMBytes / 4), map, tl.col0, tl.row0 + k * kTcK, tl.worker, m_full + s);
        }
      }
    }
    if (!ok && lane == 0)
      for (uint32_t it = kc > (uint32_t)S::kMStages ? kc - S::kMStages : 0; it < kc; ++it)
        drain(m_full + it % S::kMStages, (it / S::kMStages) & 1, abort_flag);
  } else if (warp == 1) {
    // ---- B loader: rows [row0 + 32 k, +32) of the stacked P_bar terms
    uint32_t kc = 0;
    bool ok = true;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      const Tile tl = tiles[ti];
      const uint8_t* map = maps + ((size_t)tl.layer * kTcMapsPerLayer + 1) * kTcMapBytes;
      const int nslots = tile_stages(tl.nrows) / kTcPair;
      for (int k = 0; k < nslots; ++k, ++kc) {            // kc counts slots here
        const int s = kc % S::kAB;
        if (!warp_wait(ab_empty + s, ((kc / S::kAB) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        if (lane == 0) {
          mbar_arrive_expect_tx(ab_full + s, kTcPair * S::kBBytes);
#pragma unroll
          for (int h = 0; h < kTcPair; ++h)
            tma_load_2d(bring + (size_t)(s * kTcPair + h) * S::kBStride, map, tl.row0 + (k * kTcPair + h) * kTcK, 0, ab_full + s);
        }
      }
    }
    if (!ok && lane == 0)
      for (uint32_t it = kc > (uint32_t)S::kAB ? kc - S::kAB : 0; it < kc; ++it) drain(ab_full + it % S::kAB, (it / S::kAB) & 1, abort_flag);
  } else if (warp == 2) {
    // ---- MMA issue: one thread
    if (lane == 0) {
      uint32_t kc = 0, tseq = 0;
      bool ok = true;
      const uint32_t idesc = tc_idesc_bf16(S::kN);
      const uint64_t bdesc0 = tc_desc_sw128(smem_u32(bring));     // descriptors of the other stages: + bytes / 16
      for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x, ++tseq) {
        const int nslots = tile_stages(tiles[ti].nrows) / kTcPair;
        const uint32_t db = S::kDBufs == 2 ? (tseq & 1) : 0;
        const uint32_t dcol = tmem + db * S::kDStride;
        const uint32_t dpar = S::kDBufs == 2 ? ((tseq >> 1) & 1) : (tseq & 1);
        if (!thread_wait(d_empty + db, dpar ^ 1, abort_flag)) { ok = false; break; }
        for (int k = 0; k < nslots; ++k, ++kc) {            // kc counts slots here
          const int s = kc % S::kAB;
          if (!thread_wait(ab_full + s, (kc / S::kAB) & 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t bd0 = bdesc0 + (uint64_t)((s * kTcPair * S::kBStride) >> 4);
          const uint32_t acol = tmem + S::kACol0 + s * kTcSlotK;
#pragma unroll
          for (int h = 0; h < kTcPair; ++h)
#pragma unroll
            for (int ks = 0; ks < kTcK / 8; ++ks)
              tc_mma_bf16_ts(dcol, acol + h * kTcK + ks * 8, bd0 + (uint64_t)((h * S::kBStride + ks * 32) >> 4), idesc,
                             (k > 0 || h > 0 || ks > 0) ? 1u : 0u);
          tc_commit(ab_empty + s);
          if (k == nslots - 1) tc_commit(d_full + db);
        }
      }
      // every MMA issued so far must have completed before tensor memory is released
      tc_commit(fin);
      drain(fin, 0, abort_flag);
    }
    __syncwarp();
  } else if (warp >= 4 && warp < 8) {
    // ---- epilogue: Q_w[col][j] = sum over the three N blocks of D[col][t RP + j]
    uint32_t tseq = 0;
    const int q = warp & 3;
    for (int ti = blockIdx.x; ti < ntiles; ti += gridDim.x, ++tseq) {
      const Tile tl = tiles[ti];
      const LayerDev& L = t.layers[tl.layer];
      const uint32_t db = S::kDBufs == 2 ? (tseq & 1) : 0;
      const uint32_t dpar = S::kDBufs == 2 ? ((tseq >> 1) & 1) : (tseq & 1);
      if (!warp_wait(d_full + db, dpar, abort_flag, lane)) break;
      tc_fence_after();
      const uint32_t taddr = tmem + ((uint32_t)(32 * q) << 16) + db * S::kDStride;
      const int col = tl.col0 + 32 * q + lane;
      float* dst = L.Qpart + (((size_t)tl.worker * L.nrb + tl.part) * L.m + (size_t)min(col, L.m - 1)) * RP;
      float vmax = 0.f;           // max |Q_w| over this thread's row of Q; a NaN is dropped here and reported below
      float zsum = 0.f;           // sum of 0 * value: not zero (a NaN) once a value is not finite
#pragma unroll
      for (int j0 = 0; j0 < RP; j0 += 16) {
        uint32_t a[16], b[16], c[16];
        tc_ld16(taddr + j0, a);
        tc_ld16(taddr + RP + j0, b);
        tc_ld16(taddr + 2 * RP + j0, c);
        tc_wait_ld();
        if (j0 + 16 >= RP) {      // the accumulator is in registers: the MMA thread may have it back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(d_empty + db);
        }
        if (col < L.m) {
#pragma unroll
          for (int j = 0; j < 16; j += 4) {
            float4 o;
            o.x = (__uint_as_float(c[j]) + __uint_as_float(b[j])) + __uint_as_float(a[j]);
            o.y = (__uint_as_float(c[j + 1]) + __uint_as_float(b[j + 1])) + __uint_as_float(a[j + 1]);
            o.z = (__uint_as_float(c[j + 2]) + __uint_as_float(b[j + 2])) + __uint_as_float(a[j + 2]);
            o.w = (__uint_as_float(c[j + 3]) + __uint_as_float(b[j + 3])) + __uint_as_float(a[j + 3]);
            *reinterpret_cast<float4*>(dst + j0 + j) = o;
            vmax = fmaxf(fmaxf(vmax, fmaxf(fabsf(o.x), fabsf(o.y))), fmaxf(fabsf(o.z), fabsf(o.w)));
            zsum = fmaf(0.f, o.x, fmaf(0.f, o.y, fmaf(0.f, o.z, fmaf(0.f, o.w, zsum))));
          }
        }
      }
      const bool bad = !(zsum == 0.f);
      if (L.qfused) {
        // the tile's 128 columns of M are one block of 128 rows of Q and this is the whole sum (one row chunk): the
        // block's maximum, which q_reduce would find, is taken here (non-negative floats order like their bits)
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, o));
        if (lane == 0) atomicMax(reinterpret_cast<int*>(L.maxq) + (size_t)tl.worker * L.nqb + tl.col0 / kFactorBlockRows, __float_as_int(vmax));
        if (bad) atomicOr(&t.status[tl.layer], 8u);
      }
    }
  } else if (warp >= 8) {
    // ---- consumers: M piece -> registers (lane = column) -> bf16 pair -> tensor memory
    const int g = (warp - 8) >> 2, q = warp & 3;
    uint32_t kc = 0;
    bool ok = true;
    const uint32_t lane_base = tmem + ((uint32_t)(32 * q) << 16) + S::kACol0;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      const int nk = tile_stages(tiles[ti].nrows);
      for (int k = 0; k < nk; ++k, ++kc) {
        if ((int)(kc % kTcGroups) != g) continue;
        const int s = kc % S::kMStages;
        const uint32_t slot = kc / kTcPair, ab = slot % S::kAB;
        // The slot's previous piece may have been another group's.  A barrier tells its phases apart by parity
        // alone, so this group first makes sure that piece has been taken (then its copy had landed and the
        // barrier below is in this piece's phase); asked before that, the barrier would answer for the phase
        // before, and pieces do not always land in the order they were asked for.
        if (!warp_wait(m_empty + s, ((kc / S::kMStages) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        if (!warp_wait(m_full + s, (kc / S::kMStages) & 1, abort_flag, lane)) { ok = false; break; }
        const float* src = mring + (size_t)s * (kTcMBytes / 4) + 32 * q + lane;
        uint32_t v[32];
#pragma unroll
        for (int kk = 0; kk < kTcK; ++kk) v[kk] = __float_as_uint(src[kk * kTcCols]);
        __syncwarp();
        if (lane == 0) mbar_arrive(m_empty + s);
#pragma unroll
        for (int kk = 0; kk < kTcK; ++kk) {
          const uint32_t a1 = v[kk] & 0xffff0000u;                              // bf16 by truncation, as fp32 bits
          const float r = __uint_as_float(v[kk]) - __uint_as_float(a1);         // exact
          const __nv_bfloat16 a2 = __float2bfloat16_rn(r);
          v[kk] = a1 | (uint32_t)__bfloat16_as_ushort(a2);                      // a1 in the high half, a2 in the low half
        }
        if (!warp_wait(ab_empty + ab, ((slot / S::kAB) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        tc_fence_after();
        tc_st32(lane_base + ab * kTcSlotK + (kc % kTcPair) * kTcK, v);
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(ab_full + ab);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort_flag && ntiles > 0) report_timeout(t, tiles[blockIdx.x < ntiles ? blockIdx.x : 0].layer);
  if (warp == 2)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)S::kTmemCols) : "memory");
}

// ---------------------------------------------------------------------------------------
// Pass 1 on the tensor core (P_w = M_w Q with M = G + E, Alg. 1; M is written over E).
//
// A tile is 128 rows of one worker's layer over a chunk of columns; the rows are the M extent
// of the MMA (TMEM lane = row), the columns the K extent, 32 per stage.  The HBM traffic per
// element is three times that of pass 2 (read G, read E, write M), so the tensor core has
// slack and the product keeps fp32 accuracy: tf32 operands, m = hi + lo with hi the truncation
// the hardware applies to the fp32 container and lo = m - hi, and per k-step
//   D[:, 0:2RP) += A_hi [Q_hi ; Q_lo]^T ,   D[:, 0:RP) += A_lo Q_hi^T
// (Q^T and its tf32 remainders are kept as 2 RP rows in global memory).  The epilogue adds the
// two halves of D.
//
// Stage of the ring: the 128 x 32 piece of E by TMA (128-byte swizzle: a thread reading its own
// row touches every bank once per quarter warp) and the same piece of G, also by TMA, through a
// tensor map of the caller's tensor that the host encodes when it first meets a set of gradient
// pointers (kept beside the pointer table; rows and columns past the layer are zero-filled).  A warp
// that fetched G with cp.async instead spent two thirds of the pass issuing those copies.  A consumer thread adds its row of the two pieces, puts m back into the
// E piece (a storer thread sends it to global memory with a TMA tensor store) and writes hi and
// lo to TMEM.
// ---------------------------------------------------------------------------------------
constexpr int kT1Stages = 5;          // ring of (G, E) pieces, 2 x 16 KB each
constexpr int kT1AB = 4;              // ring of A (TMEM, hi + lo: 64 columns) and B (shared memory) buffers
constexpr uint32_t kT1PieceBytes = 128 * 128;   // 128 rows x 32 fp32

__device__ __forceinline__ void tc_mma_tf32_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n}"
               ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Instruction descriptor: tf32 x tf32 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t tc_idesc_tf32(int n) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const void* tmap, int x, int y, int z, const void* smem_src) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
               ::"l"(tmap), "r"(x), "r"(y), "r"(z), "r"(smem_u32(smem_src)) : "memory");
}
// the executing thread's cp.async copies issued so far arrive on `bar` when they have landed
__device__ __forceinline__ void cp_async_arrive(uint64_t* bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

template <int RP>
struct Pass1Cfg {
  static constexpr int kDStride = 2 * RP <= 64 ? 64 : (2 * RP <= 128 ? 128 : 256);
  static constexpr int kACol0 = 2 * kDStride;
  static constexpr int kTmemCols = 512;
  static constexpr uint32_t kBBytes = 2 * RP * 128;                      // Q_hi rows, then Q_lo rows, 32 columns
  static constexpr int kStages = kT1Stages;                               // ring of (G, E) pieces
  static constexpr uint32_t kBOff = kStages * 2 * kT1PieceBytes;
  static constexpr uint32_t kBarOff = kBOff + kT1AB * kBBytes;
  static constexpr int kBars = 3 * kStages + 2 * kT1AB + 2 + 2 + 1 + 2 * kTqDepth;   // ..., fin, tile queue
  static constexpr uint32_t kTotal = kBarOff + kBars * 8 + 16 + 4 * kTqDepth + 1024;
  static_assert(kACol0 + kT1AB * 64 <= 512, "tensor memory");
  static_assert(kBBytes % 1024 == 0, "B stages stay 1024-byte aligned");
  static_assert(kTotal <= 227 * 1024, "shared memory");
  static_assert(kStages < 2 * kT1AB, "a consumer must not get two turns of the operand ring ahead (see Pass2Cfg)");
};

template <int RP>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_pass1_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles, int* __restrict__ sched, const uint8_t* __restrict__ maps) {
  pdl_wait();
  clear_status_words(t);
  using S = Pass1Cfg<RP>;
  constexpr int kT1Stages = S::kStages;          // this rank's ring depth
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* bring = base + S::kBOff;
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + S::kBarOff);
  uint64_t* ge_full = bars;                      // [kT1Stages] G and E landed
  uint64_t* m_ready = ge_full + kT1Stages;       // [kT1Stages] consumers have put m into the E piece
  uint64_t* ge_empty = m_ready + kT1Stages;      // [kT1Stages] the store of m has read the piece: refill
  uint64_t* ab_full = ge_empty + kT1Stages;      // [kT1AB] A written to TMEM (4 warps) and B landed
  uint64_t* ab_empty = ab_full + kT1AB;          // [kT1AB] the MMAs that read buffer i have completed
  uint64_t* d_full = ab_empty + kT1AB;           // [2]
  uint64_t* d_empty = d_full + 2;                // [2]
  uint64_t* fin = d_empty + 2;                   // [1]
  uint64_t* q_full = fin + 1;                    // [kTqDepth] tile queue
  uint64_t* q_empty = q_full + kTqDepth;         // [kTqDepth]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(q_empty + kTqDepth);
  uint32_t* tmem_slot = const_cast<uint32_t*>(reinterpret_cast<volatile uint32_t*>(abort_flag)) + 2;   // after the abort flag and the wait limit
  const TileQueue tq{q_full, q_empty, reinterpret_cast<volatile int*>(tmem_slot + 2)};

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < kT1Stages; ++s) { mbar_init(ge_full + s, 1); mbar_init(m_ready + s, 4); mbar_init(ge_empty + s, 1); }
    for (int s = 0; s < kT1AB; ++s) { mbar_init(ab_full + s, 5); mbar_init(ab_empty + s, 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(d_full + s, 1); mbar_init(d_empty + s, 4); }
    mbar_init(fin, 1);
    // readers of the tile queue: B loader, MMA thread, storer, 4 epilogue warps, 12 consumer warps
    for (int s = 0; s < kTqDepth; ++s) { mbar_init(q_full + s, 1); mbar_init(q_empty + s, 3 + 4 + 4 * kTcGroups); }
    wait_ctl_init(abort_flag, t.wait_limit);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)S::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  auto g_piece = [&](int s) { return base + (size_t)s * 2 * kT1PieceBytes; };
  auto e_piece = [&](int s) { return base + (size_t)s * 2 * kT1PieceBytes + kT1PieceBytes; };

  if (warp == 0) {
    // ---- loader: the piece of E and the same piece of this worker's G, two tensor copies
    uint32_t kc = 0, qs = 0;
    bool ok = true;
    int ti = (int)blockIdx.x < ntiles ? (int)blockIdx.x : kTqEnd;
    for (;; ++qs) {
      int put = 1, drawn = kTqEnd;
      if (lane == 0) {
        put = tq_put(tq, qs, ti, abort_flag) ? 1 : 0;
        if (put && ti != kTqEnd) drawn = tq_draw(sched, ntiles);        // the tile after this one: the answer comes meanwhile
      }
      if (!__shfl_sync(0xffffffffu, put, 0)) { ok = false; break; }
      if (ti == kTqEnd) break;
      const Tile tl = tiles[ti];
      const LayerDev& L = t.layers[tl.layer];
      const uint8_t* map = maps + ((size_t)tl.layer * kTcMapsPerLayer + 2) * kTcMapBytes;
      const uint8_t* gmap = t.gmaps + ((size_t)tl.layer * t.W + tl.worker) * kTcMapBytes;   // this worker's gradient
      const int nk = (tl.ncols + kTcK - 1) / kTcK;
      for (int k = 0; k < nk; ++k, ++kc) {
        const int s = kc % kT1Stages;
        if (!warp_wait(ge_empty + s, ((kc / kT1Stages) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        if (test_skips_stage(t, 1, kc)) continue;     // test support: this piece is not fetched, its waiters give up
        const int c0 = tl.col0 + k * kTcK;
        if (lane == 0) {
          mbar_arrive_expect_tx(ge_full + s, 2 * kT1PieceBytes);
          tma_load_3d(e_piece(s), map, c0, tl.row0, tl.worker, ge_full + s);
          tma_load_2d(g_piece(s), gmap, c0, tl.row0, ge_full + s);
        }
      }
      if (!ok) break;
      ti = __shfl_sync(0xffffffffu, drawn, 0);
    }
    if (!ok && lane == 0)
      for (uint32_t it = kc > (uint32_t)kT1Stages ? kc - kT1Stages : 0; it < kc; ++it)
        drain(ge_full + it % kT1Stages, (it / kT1Stages) & 1, abort_flag);
  } else if (warp == 1) {
    // ---- B loader: columns [c0, c0 + 32) of Q^T and of its remainders
    uint32_t kc = 0;
    bool ok = true;
    for (uint32_t qs = 0; ok; ++qs) {
      const int ti = tq_take_warp(tq, qs, abort_flag, lane);
      if (ti < 0) { ok = ti == kTqEnd; break; }
      const Tile tl = tiles[ti];
      const uint8_t* map = maps + ((size_t)tl.layer * kTcMapsPerLayer + 3) * kTcMapBytes;
      const int nk = (tl.ncols + kTcK - 1) / kTcK;
      for (int k = 0; k < nk; ++k, ++kc) {
        const int s = kc % kT1AB;
        if (!warp_wait(ab_empty + s, ((kc / kT1AB) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        if (lane == 0) {
          mbar_arrive_expect_tx(ab_full + s, S::kBBytes);
          tma_load_2d(bring + (size_t)s * S::kBBytes, map, tl.col0 + k * kTcK, 0, ab_full + s);
        }
      }
    }
    if (!ok && lane == 0)
      for (uint32_t it = kc > (uint32_t)kT1AB ? kc - kT1AB : 0; it < kc; ++it) drain(ab_full + it % kT1AB, (it / kT1AB) & 1, abort_flag);
  } else if (warp == 2) {
    // ---- MMA issue: one thread
    if (lane == 0) {
      uint32_t kc = 0, tseq = 0;
      bool ok = true;
      const uint32_t idesc2 = tc_idesc_tf32(2 * RP), idesc1 = tc_idesc_tf32(RP);
      const uint64_t bdesc0 = tc_desc_sw128(smem_u32(bring));
      for (; ok; ++tseq) {
        const int ti = tq_take(tq, tseq, abort_flag);
        if (ti < 0) { ok = ti == kTqEnd; break; }
        const int nk = (tiles[ti].ncols + kTcK - 1) / kTcK;
        const uint32_t db = tseq & 1;
        const uint32_t dcol = tmem + db * S::kDStride;
        if (!thread_wait(d_empty + db, ((tseq >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
        for (int k = 0; k < nk; ++k, ++kc) {
          const int s = kc % kT1AB;
          if (!thread_wait(ab_full + s, (kc / kT1AB) & 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t bd0 = bdesc0 + (uint64_t)((s * S::kBBytes) >> 4);
          const uint32_t acol = tmem + S::kACol0 + s * 64;
#pragma unroll
          for (int ks = 0; ks < kTcK / 8; ++ks) {
            tc_mma_tf32_ts(dcol, acol + ks * 8, bd0 + (uint64_t)((ks * 32) >> 4), idesc2, (k > 0 || ks > 0) ? 1u : 0u);
            tc_mma_tf32_ts(dcol, acol + 32 + ks * 8, bd0 + (uint64_t)((ks * 32) >> 4), idesc1, 1u);
          }
          tc_commit(ab_empty + s);
          if (k == nk - 1) tc_commit(d_full + db);
        }
      }
      tc_commit(fin);
      drain(fin, 0, abort_flag);
    }
    __syncwarp();
  } else if (warp == 3) {
    // ---- storer: m pieces back to global memory (over E)
    uint32_t kc = 0;
    bool ok = true;
    for (uint32_t qs = 0; ok; ++qs) {
      const int ti = tq_take_warp(tq, qs, abort_flag, lane);
      if (ti < 0) { ok = ti == kTqEnd; break; }
      const Tile tl = tiles[ti];
      const uint8_t* map = maps + ((size_t)tl.layer * kTcMapsPerLayer + 2) * kTcMapBytes;
      const int nk = (tl.ncols + kTcK - 1) / kTcK;
      for (int k = 0; k < nk; ++k, ++kc) {
        const int s = kc % kT1Stages;
        if (!warp_wait(m_ready + s, (kc / kT1Stages) & 1, abort_flag, lane)) { ok = false; break; }
        if (lane == 0) {
          tma_store_3d(map, tl.col0 + k * kTcK, tl.row0, tl.worker, e_piece(s));
          bulk_commit();
          // one store stays in flight: the stage of the store before this one is free once that one has been read
          if (kc > 0) {
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            mbar_arrive(ge_empty + (kc - 1) % kT1Stages);
          }
        }
        __syncwarp();
      }
    }
    if (lane == 0) {
      bulk_wait_read0();
      if (ok && kc > 0) mbar_arrive(ge_empty + (kc - 1) % kT1Stages);
      bulk_wait_all0();
    }
  } else if (warp < 8) {
    // ---- epilogue: P_part[row][j] = D[row][j] + D[row][RP + j]
    uint32_t tseq = 0;
    const int q = warp & 3;
    for (;; ++tseq) {
      const int ti = tq_take_warp(tq, tseq, abort_flag, lane);
      if (ti < 0) break;
      const Tile tl = tiles[ti];
      const LayerDev& L = t.layers[tl.layer];
      const uint32_t db = tseq & 1;
      if (!warp_wait(d_full + db, (tseq >> 1) & 1, abort_flag, lane)) break;
      tc_fence_after();
      const uint32_t taddr = tmem + ((uint32_t)(32 * q) << 16) + db * S::kDStride;
      const int row = tl.row0 + 32 * q + lane;
      float* dst = L.Ppart + (((size_t)tl.worker * L.ncc + tl.part) * L.n + (size_t)min(row, L.n - 1)) * RP;
#pragma unroll
      for (int j0 = 0; j0 < RP; j0 += 16) {
        uint32_t a[16], b[16];
        tc_ld16(taddr + j0, a);
        tc_ld16(taddr + RP + j0, b);
        tc_wait_ld();
        if (row < L.n) {
#pragma unroll
          for (int j = 0; j < 16; j += 4)
            *reinterpret_cast<float4*>(dst + j0 + j) =
                make_float4(__uint_as_float(a[j]) + __uint_as_float(b[j]), __uint_as_float(a[j + 1]) + __uint_as_float(b[j + 1]),
                            __uint_as_float(a[j + 2]) + __uint_as_float(b[j + 2]), __uint_as_float(a[j + 3]) + __uint_as_float(b[j + 3]));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(d_empty + db);
    }
  } else {
    // ---- consumers: lane = row; m = g + e -> E piece (for the store) and hi / lo -> tensor memory
    const int g = (warp - 8) >> 2, q = warp & 3;
    uint32_t kc = 0;
    bool ok = true;
    const uint32_t lane_base = tmem + ((uint32_t)(32 * q) << 16) + S::kACol0;
    const int row = 32 * q + lane;
    for (uint32_t qs = 0; ok; ++qs) {
      const int ti = tq_take_warp(tq, qs, abort_flag, lane);
      if (ti < 0) { ok = ti == kTqEnd; break; }
      const int nk = (tiles[ti].ncols + kTcK - 1) / kTcK;
      for (int k = 0; k < nk; ++k, ++kc) {
        if ((int)(kc % kTcGroups) != g) continue;
        const int s = kc % kT1Stages, ab = kc % kT1AB;
        // first the slot's previous piece must have been taken, by whichever group had it (see pass 2)
        if (!warp_wait(m_ready + s, ((kc / kT1Stages) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        if (!warp_wait(ge_full + s, (kc / kT1Stages) & 1, abort_flag, lane)) { ok = false; break; }
        const uint8_t* gp = g_piece(s) + row * 128;
        uint8_t* ep = e_piece(s) + row * 128;
        uint32_t v[32];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const int off = (c ^ (row & 7)) << 4;
          const float4 g4 = *reinterpret_cast<const float4*>(gp + off);
          float4 e4 = *reinterpret_cast<const float4*>(ep + off);
          e4.x += g4.x; e4.y += g4.y; e4.z += g4.z; e4.w += g4.w;
          *reinterpret_cast<float4*>(ep + off) = e4;
          v[4 * c] = __float_as_uint(e4.x); v[4 * c + 1] = __float_as_uint(e4.y);
          v[4 * c + 2] = __float_as_uint(e4.z); v[4 * c + 3] = __float_as_uint(e4.w);
        }
        fence_async_smem();                       // the TMA store reads what was just written
        __syncwarp();
        if (lane == 0) mbar_arrive(m_ready + s);
        if (!warp_wait(ab_empty + ab, ((kc / kT1AB) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        tc_fence_after();
        tc_st32(lane_base + ab * 64, v);
#pragma unroll
        for (int kk = 0; kk < 32; ++kk) {
          const float x = __uint_as_float(v[kk]);
          v[kk] = __float_as_uint(x - __uint_as_float(v[kk] & 0xffffe000u));
        }
        tc_st32(lane_base + ab * 64 + 32, v);
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(ab_full + ab);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort_flag && ntiles > 0) report_timeout(t, tiles[min((int)blockIdx.x, ntiles - 1)].layer);
  if (tid == 0) tq_leave(sched);
  if (warp == 2)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)S::kTmemCols) : "memory");
}

// ---------------------------------------------------------------------------------------
// Pass 3 on the tensor core (G_hat = P_bar Q_bar^T, E_w = M_w - G_hat, Alg. 1; optional model
// update).  A tile is 128 rows x 128 columns of one layer, for a range of workers [worker, part).  Once per tile the
// accumulator D = G_hat tile is formed from the factors: both operands come from shared memory,
// K-major, as rows of kCat = 3 RP (padded to a multiple of 32) tf32 values
//   P side: [P_bar | P_bar | P_bar_lo | 0]      Q side: [Q_bar | Q_bar_lo | Q_bar | 0]
// (lo = the remainder after the truncation to tf32 the hardware applies), so that one K loop
// yields hi*hi + hi*lo + lo*hi.  Then, for every worker, the 128 x 128 piece of M streams through
// a ring in four 128 x 32 pieces (TMA, 128-byte swizzle); a consumer thread (lane = row) reads its
// row of G_hat from tensor memory, subtracts, puts E back into the piece (a storer thread sends
// it to global memory with a TMA tensor store); the warpgroup that meets worker 0 also writes
// G_hat and applies the model update.
// ---------------------------------------------------------------------------------------
constexpr int kT3Stages = 8;          // ring of M pieces, 16 KB each
constexpr int kT3Groups = 4;          // consumer warpgroups (warps 4..19)

__device__ __forceinline__ void tc_mma_tf32_ss(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
               ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

template <int RP>
struct Pass3Cfg {
  static constexpr int kCat = (3 * RP + 31) / 32 * 32;                   // K extent of the factor product
  static constexpr int kHalves = RP <= 32 ? 1 : 2;                       // the operands come in this many K slices, one after
                                                                         // the other through the same buffer (rank 64: 2 x 96)
  static constexpr int kSub = kCat / 32 / kHalves;                       // 128-byte sub-tiles per operand slice
  static constexpr uint32_t kOpBytes = kSub * kT1PieceBytes;             // one operand slice: kSub pieces of 128 rows x 32
  static constexpr int kStages = kT3Stages;                               // ring of M pieces
  static constexpr uint32_t kOpOff = kStages * kT1PieceBytes;
  static constexpr uint32_t kBarOff = kOpOff + 2 * kOpBytes;
  static constexpr int kBars = 3 * kStages + 2 + 2 + 2 + 2 + 1 + 2 * kTqDepth;   // m_full, e_ready, m_empty; op_full, op_empty, d_full, d_empty (2 each); fin; tile queue
  static constexpr uint32_t kTotal = kBarOff + kBars * 8 + 16 + 4 * kTqDepth + 1024;
  static constexpr int kTmemCols = 256;                                  // two accumulators of 128 columns
  static_assert((kCat / 32) % kHalves == 0 && kTotal <= 227 * 1024, "operand slices, shared memory");
};

template <int RP>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_pass3_kernel(Tables t, const Tile* __restrict__ tiles, int ntiles, int* __restrict__ sched, const uint8_t* __restrict__ maps) {
  pdl_wait();
  using S = Pass3Cfg<RP>;
  constexpr int kT3Stages = S::kStages;          // this rank's ring depth
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* opa = base + S::kOpOff;               // P side
  uint8_t* opb = opa + S::kOpBytes;              // Q side
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + S::kBarOff);
  uint64_t* m_full = bars;                       // [kT3Stages] piece of M landed
  uint64_t* e_ready = m_full + kT3Stages;        // [kT3Stages] consumers have put E into the piece
  uint64_t* m_empty = e_ready + kT3Stages;       // [kT3Stages] the store of E has read the piece
  uint64_t* op_full = m_empty + kT3Stages;       // [1] operands of the tile landed   (+1 spare)
  uint64_t* op_empty = op_full + 2;              // [1] the tile's MMAs have completed (+1 spare)
  uint64_t* d_full = op_empty + 2;               // [2]
  uint64_t* d_empty = d_full + 2;                // [2] all 16 consumer warps are past the tile
  uint64_t* fin = d_empty + 2;
  uint64_t* q_full = fin + 1;                    // [kTqDepth] tile queue
  uint64_t* q_empty = q_full + kTqDepth;         // [kTqDepth]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(q_empty + kTqDepth);
  uint32_t* tmem_slot = const_cast<uint32_t*>(reinterpret_cast<volatile uint32_t*>(abort_flag)) + 2;   // after the abort flag and the wait limit
  const TileQueue tq{q_full, q_empty, reinterpret_cast<volatile int*>(tmem_slot + 2)};

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < kT3Stages; ++s) { mbar_init(m_full + s, 1); mbar_init(e_ready + s, 4); mbar_init(m_empty + s, 1); }
    mbar_init(op_full, 1); mbar_init(op_empty, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(d_full + s, 1); mbar_init(d_empty + s, 4 * kT3Groups); }
    mbar_init(fin, 1);
    // readers of the tile queue: operand loader, MMA thread, storer, 16 consumer warps
    for (int s = 0; s < kTqDepth; ++s) { mbar_init(q_full + s, 1); mbar_init(q_empty + s, 3 + 4 * kT3Groups); }
    wait_ctl_init(abort_flag, t.wait_limit);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)S::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  auto piece = [&](int s) { return base + (size_t)s * kT1PieceBytes; };
  auto pieces_of = [](const Tile& tl) { return (tl.ncols + kTcK - 1) / kTcK; };

  if (warp == 0) {
    // ---- M loader
    // The queue runs one entry ahead of the loads: while this warp fetches the pieces of one entry, the operand
    // loader and the MMA thread already form G_hat of the next (two accumulators), so that the consumers find it
    // ready.  The first two entries are fixed (tiles b and b + gridDim.x), the counter hands out the rest.
    uint32_t kc = 0, qs = 0;
    bool ok = true;
    int ti = (int)blockIdx.x < ntiles ? (int)blockIdx.x : kTqEnd;
    int nxt = ti != kTqEnd && (int)(blockIdx.x + gridDim.x) < ntiles ? (int)(blockIdx.x + gridDim.x) : kTqEnd;
    {
      int put = 1;
      if (lane == 0) put = tq_put(tq, qs, ti, abort_flag) ? 1 : 0;
      ++qs;
      if (!__shfl_sync(0xffffffffu, put, 0)) { ok = false; ti = kTqEnd; }
    }
    for (; ti != kTqEnd; ++qs) {
      int put = 1, drawn = kTqEnd;
      if (lane == 0) {
        put = tq_put(tq, qs, nxt, abort_flag) ? 1 : 0;
        if (put && nxt != kTqEnd) drawn = tq_draw(sched, ntiles, 2);    // the entry after the next: the answer comes meanwhile
      }
      if (!__shfl_sync(0xffffffffu, put, 0)) { ok = false; break; }
      const Tile tl = tiles[ti];
      const uint8_t* map = maps + ((size_t)tl.layer * kTcMapsPerLayer + 2) * kTcMapBytes;
      const int np = pieces_of(tl);
      for (int w = tl.worker; w < tl.part && ok; ++w)
        for (int pc = 0; pc < np; ++pc, ++kc) {
          const int s = kc % kT3Stages;
          if (!warp_wait(m_empty + s, ((kc / kT3Stages) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
          if (test_skips_stage(t, 3, kc)) continue;   // test support, as in pass 1
          if (lane == 0) {
            mbar_arrive_expect_tx(m_full + s, kT1PieceBytes);
            tma_load_3d(piece(s), map, tl.col0 + pc * kTcK, tl.row0, w, m_full + s);
          }
        }
      if (!ok) break;
      ti = nxt;
      nxt = __shfl_sync(0xffffffffu, drawn, 0);
    }
    if (!ok && lane == 0)
      for (uint32_t it = kc > (uint32_t)kT3Stages ? kc - kT3Stages : 0; it < kc; ++it)
        drain(m_full + it % kT3Stages, (it / kT3Stages) & 1, abort_flag);
  } else if (warp == 1) {
    // ---- operand loader: the tile's rows of the stacked P_bar terms and its columns' rows of the Q_bar terms
    uint32_t oseq = 0;                      // operand slices loaded so far (kHalves per tile)
    bool ok = true;
    for (uint32_t qs = 0; ok; ++qs) {
      const int ti = tq_take_warp(tq, qs, abort_flag, lane);
      if (ti < 0) { ok = ti == kTqEnd; break; }
      const Tile tl = tiles[ti];
      const uint8_t* mapp = maps + ((size_t)tl.layer * kTcMapsPerLayer + 4) * kTcMapBytes;
      const uint8_t* mapq = maps + ((size_t)tl.layer * kTcMapsPerLayer + 5) * kTcMapBytes;
      for (int h = 0; h < S::kHalves; ++h, ++oseq) {
        if (!warp_wait(op_empty, (oseq & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        if (lane == 0) {
          mbar_arrive_expect_tx(op_full, 2 * S::kOpBytes);
#pragma unroll
          for (int kt = 0; kt < S::kSub; ++kt) {
            tma_load_2d(opa + (size_t)kt * kT1PieceBytes, mapp, (h * S::kSub + kt) * 32, tl.row0, op_full);
            tma_load_2d(opb + (size_t)kt * kT1PieceBytes, mapq, (h * S::kSub + kt) * 32, tl.col0, op_full);
          }
        }
      }
    }
    if (!ok && lane == 0 && oseq > 0) drain(op_full, (oseq - 1) & 1, abort_flag);
  } else if (warp == 2) {
    // ---- MMA issue: one thread, once per tile
    if (lane == 0) {
      uint32_t tseq = 0, oseq = 0;
      bool ok = true;
      const uint32_t idesc = tc_idesc_tf32(128);
      const uint64_t adesc0 = tc_desc_sw128(smem_u32(opa)), bdesc0 = tc_desc_sw128(smem_u32(opb));
      for (; ok; ++tseq) {
        const int ti = tq_take(tq, tseq, abort_flag);
        if (ti < 0) { ok = ti == kTqEnd; break; }
        const uint32_t db = tseq & 1;
        if (!thread_wait(d_empty + db, ((tseq >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
        for (int h = 0; h < S::kHalves && ok; ++h, ++oseq) {
          if (!thread_wait(op_full, oseq & 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int kt = 0; kt < S::kSub; ++kt)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t off = (uint64_t)((kt * kT1PieceBytes + ks * 32) >> 4);
              tc_mma_tf32_ss(tmem + db * 128, adesc0 + off, bdesc0 + off, idesc, (h > 0 || kt > 0 || ks > 0) ? 1u : 0u);
            }
          tc_commit(op_empty);            // the slice's buffer may be refilled once these MMAs have read it
        }
        if (ok) tc_commit(d_full + db);
      }
      tc_commit(fin);
      drain(fin, 0, abort_flag);
    }
    __syncwarp();
  } else if (warp == 3) {
    // ---- storer: E pieces back to global memory
    uint32_t kc = 0;
    bool ok = true;
    for (uint32_t qs = 0; ok; ++qs) {
      const int ti = tq_take_warp(tq, qs, abort_flag, lane);
      if (ti < 0) { ok = ti == kTqEnd; break; }
      const Tile tl = tiles[ti];
      const uint8_t* map = maps + ((size_t)tl.layer * kTcMapsPerLayer + 2) * kTcMapBytes;
      const int np = pieces_of(tl);
      for (int w = tl.worker; w < tl.part && ok; ++w)
        for (int pc = 0; pc < np; ++pc, ++kc) {
          const int s = kc % kT3Stages;
          if (!warp_wait(e_ready + s, (kc / kT3Stages) & 1, abort_flag, lane)) { ok = false; break; }
          if (lane == 0) {
            tma_store_3d(map, tl.col0 + pc * kTcK, tl.row0, w, piece(s));
            bulk_commit();
            if (kc > 0) {
              asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
              mbar_arrive(m_empty + (kc - 1) % kT3Stages);
            }
          }
          __syncwarp();
        }
    }
    if (lane == 0) {
      bulk_wait_read0();
      if (ok && kc > 0) mbar_arrive(m_empty + (kc - 1) % kT3Stages);
      bulk_wait_all0();
    }
  } else {
    // ---- consumers (warps 4..19): lane = row
    const int g = (warp - 4) >> 2, q = warp & 3;
    uint32_t kc = 0, tseq = 0;
    bool ok = true;
    const int row_in_tile = 32 * q + lane;
    for (; ok; ++tseq) {
      const int ti = tq_take_warp(tq, tseq, abort_flag, lane);
      if (ti < 0) { ok = ti == kTqEnd; break; }
      const Tile tl = tiles[ti];
      const LayerDev& L = t.layers[tl.layer];
      const int np = pieces_of(tl);
      const uint32_t db = tseq & 1;
      const uint32_t taddr = tmem + ((uint32_t)(32 * q) << 16) + db * 128;
      const int row = tl.row0 + row_in_tile;
      float* Gh = t.ghat[tl.layer];
      float* Wt = t.weights ? t.weights[tl.layer] : nullptr;
      // every warp waits for the tile's accumulator, also one that meets none of its pieces: its
      // arrival on d_empty below must not run ahead of the tile
      if (!warp_wait(d_full + db, (tseq >> 1) & 1, abort_flag, lane)) { ok = false; break; }
      tc_fence_after();
      for (int w = tl.worker; w < tl.part && ok; ++w)
        for (int pc = 0; pc < np; ++pc, ++kc) {
          if ((int)(kc % kT3Groups) != g) continue;
          const int s = kc % kT3Stages;
          // first the slot's previous piece must have been taken, by whichever group had it (see pass 2)
          if (!warp_wait(e_ready + s, ((kc / kT3Stages) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
          uint32_t gh[32];
          tc_ld32(taddr + pc * 32, gh);
          if (!warp_wait(m_full + s, (kc / kT3Stages) & 1, abort_flag, lane)) { tc_wait_ld(); ok = false; break; }
          tc_wait_ld();
          uint8_t* mp = piece(s) + row_in_tile * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const int off = (c ^ (row_in_tile & 7)) << 4;
            float4 m4 = *reinterpret_cast<const float4*>(mp + off);
            m4.x -= __uint_as_float(gh[4 * c]); m4.y -= __uint_as_float(gh[4 * c + 1]);
            m4.z -= __uint_as_float(gh[4 * c + 2]); m4.w -= __uint_as_float(gh[4 * c + 3]);
            *reinterpret_cast<float4*>(mp + off) = m4;
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(e_ready + s);
          if (w == 0 && row < L.n) {
            // G_hat itself (and the model update w <- w - lr * G_hat): the thread's 32 consecutive columns
            const int c0 = tl.col0 + pc * kTcK;
            const size_t o = (size_t)row * L.m + c0;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              if (c0 + 4 * c < L.m) {
                const float4 g4 = make_float4(__uint_as_float(gh[4 * c]), __uint_as_float(gh[4 * c + 1]),
                                              __uint_as_float(gh[4 * c + 2]), __uint_as_float(gh[4 * c + 3]));
                if (Gh) __stcs(reinterpret_cast<float4*>(Gh + o) + c, g4);
                if (Wt) {
                  float4* wp = reinterpret_cast<float4*>(Wt + o) + c;
                  float4 wv = __ldcs(wp);
                  wv.x = fmaf(-t.lr, g4.x, wv.x); wv.y = fmaf(-t.lr, g4.y, wv.y);
                  wv.z = fmaf(-t.lr, g4.z, wv.z); wv.w = fmaf(-t.lr, g4.w, wv.w);
                  __stcs(wp, wv);
                }
              }
            }
          }
        }
      // past the tile: this warp no longer reads its accumulator
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(d_empty + db);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort_flag && ntiles > 0) report_timeout(t, tiles[min((int)blockIdx.x, ntiles - 1)].layer);
  if (tid == 0) tq_leave(sched);
  if (warp == 2)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)S::kTmemCols) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

// Fills kTcMapsPerLayer tensor maps per layer (host memory, 128 bytes each); layers that the
// tensor-core passes do not take get zeros.
// Every map asks L2 to fetch 256 bytes around a 128-byte access: a piece is 128 rows of 128 bytes, a row's next 128
// bytes belong to the piece that is asked for next, and memory serves 256-byte requests better (pass 1 on the
// 16-worker set: 387 -> 359 us).
int tc_encode_maps(const LayerDev* layers, int n_layers, int W, int RP, void* out) {
  static_assert(sizeof(CUtensorMap) == kTcMapBytes, "tensor map size");
  std::memset(out, 0, (size_t)n_layers * kTcMapsPerLayer * kTcMapBytes);
  bool any = false;
  for (int i = 0; i < n_layers; ++i) any = any || layers[i].tc;
  if (!any) return LQSGD_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return LQSGD_ERR_CUDA;
  EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(fn);
  CUtensorMap* maps = static_cast<CUtensorMap*>(out);
  for (int i = 0; i < n_layers; ++i) {
    const LayerDev& L = layers[i];
    if (!L.tc) continue;
    {   // M (held in E) as [W][n][m]: pieces of 32 rows x 128 columns, rows past n read as zero
      const cuuint64_t dim[3] = {(cuuint64_t)L.m, (cuuint64_t)L.n, (cuuint64_t)W};
      const cuuint64_t stride[2] = {(cuuint64_t)L.m * 4, (cuuint64_t)L.n * L.m * 4};
      const cuuint32_t box[3] = {kTcCols, kTcK, 1}, es[3] = {1, 1, 1};
      if (encode(&maps[i * kTcMapsPerLayer + 0], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, L.E, dim, stride, box, es,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return LQSGD_ERR_CUDA;
    }
    {   // stacked bf16 terms of P_bar^T, [3 RP][nt] words (a bf16 value twice per word): 32 rows of P_bar
      const cuuint64_t dim[2] = {(cuuint64_t)L.nt, (cuuint64_t)(3 * RP)};
      const cuuint64_t stride[1] = {(cuuint64_t)L.nt * 4};
      const cuuint32_t box[2] = {kTcK, (cuuint32_t)(3 * RP)}, es[2] = {1, 1};
      if (encode(&maps[i * kTcMapsPerLayer + 1], CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, L.Pbt, dim, stride, box, es,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return LQSGD_ERR_CUDA;
    }
    {   // E / M as [W][n][m]: pieces of 128 rows x 32 columns, 128-byte swizzle (pass 1: load E, store M)
      const cuuint64_t dim[3] = {(cuuint64_t)L.m, (cuuint64_t)L.n, (cuuint64_t)W};
      const cuuint64_t stride[2] = {(cuuint64_t)L.m * 4, (cuuint64_t)L.n * L.m * 4};
      const cuuint32_t box[3] = {kTcK, 128, 1}, es[3] = {1, 1, 1};
      if (encode(&maps[i * kTcMapsPerLayer + 2], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, L.E, dim, stride, box, es,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return LQSGD_ERR_CUDA;
    }
    {   // stacked terms of P_bar, [n][kcat], and of Q_bar, [m][kcat]: 128 rows x 32 values (pass 3 operands)
      const cuuint32_t box[2] = {kTcK, 128}, es[2] = {1, 1};
      const cuuint64_t dimp[2] = {(cuuint64_t)L.kcat, (cuuint64_t)L.n}, dimq[2] = {(cuuint64_t)L.kcat, (cuuint64_t)L.m};
      const cuuint64_t stride[1] = {(cuuint64_t)L.kcat * 4};
      if (encode(&maps[i * kTcMapsPerLayer + 4], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, L.Pcat, dimp, stride, box, es,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
          encode(&maps[i * kTcMapsPerLayer + 5], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, L.Qcat, dimq, stride, box, es,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return LQSGD_ERR_CUDA;
    }
    {   // Q^T and its tf32 remainders, [2 RP][mt]: 32 columns of Q for all 2 RP operand rows (pass 1)
      const cuuint64_t dim[2] = {(cuuint64_t)L.mt, (cuuint64_t)(2 * RP)};
      const cuuint64_t stride[1] = {(cuuint64_t)L.mt * 4};
      const cuuint32_t box[2] = {kTcK, (cuuint32_t)(2 * RP)}, es[2] = {1, 1};
      if (encode(&maps[i * kTcMapsPerLayer + 3], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, L.Qt, dim, stride, box, es,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return LQSGD_ERR_CUDA;
    }
  }
  return LQSGD_OK;
}

// One tensor map per (layer, worker) over the caller's gradient, [n][m] fp32: pieces of 128 rows x 32 columns, 128-byte
// swizzle (pass 1).  grads: [n_layers][W] device pointers, 16-byte aligned for the layers concerned; out: [n_layers][W] maps.
int tc_encode_grad_maps(const LayerDev* layers, int n_layers, int W, const void* const* grads, void* out) {
  std::memset(out, 0, (size_t)n_layers * W * kTcMapBytes);
  static EncodeTiledFn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
      return LQSGD_ERR_CUDA;
    encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  CUtensorMap* maps = static_cast<CUtensorMap*>(out);
  for (int i = 0; i < n_layers; ++i) {
    const LayerDev& L = layers[i];
    if (!L.tc) continue;
    const cuuint64_t dim[2] = {(cuuint64_t)L.m, (cuuint64_t)L.n};
    const cuuint64_t stride[1] = {(cuuint64_t)L.m * 4};
    const cuuint32_t box[2] = {kTcK, 128}, es[2] = {1, 1};
    for (int w = 0; w < W; ++w)
      if (encode(&maps[(size_t)i * W + w], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(grads[(size_t)i * W + w]), dim, stride,
                 box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return LQSGD_ERR_CUDA;
  }
  return LQSGD_OK;
}

cudaError_t launch_tc_pass3(int RP, const Tables& t, const Tile* tiles, int ntiles, int* sched, const void* maps,
                            Launch l) {
  if (ntiles == 0) return cudaSuccess;
  auto go = [&](auto kernel, size_t smem) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_pdl(kernel, dim3(l.grid), dim3(kTcThreads), smem, l.stream, t, tiles, ntiles, sched, static_cast<const uint8_t*>(maps));
  };
  if (RP == 16) return go(tc_pass3_kernel<16>, Pass3Cfg<16>::kTotal);
  if (RP == 32) return go(tc_pass3_kernel<32>, Pass3Cfg<32>::kTotal);
  if (RP == 64) return go(tc_pass3_kernel<64>, Pass3Cfg<64>::kTotal);
  return cudaErrorInvalidValue;
}

cudaError_t launch_tc_pass1(int RP, const Tables& t, const Tile* tiles, int ntiles, int* sched, const void* maps,
                            Launch l) {
  if (ntiles == 0) return cudaSuccess;
  auto go = [&](auto kernel, size_t smem) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_pdl(kernel, dim3(l.grid), dim3(kTcThreads), smem, l.stream, t, tiles, ntiles, sched, static_cast<const uint8_t*>(maps));
  };
  if (RP == 16) return go(tc_pass1_kernel<16>, Pass1Cfg<16>::kTotal);
  if (RP == 32) return go(tc_pass1_kernel<32>, Pass1Cfg<32>::kTotal);
  if (RP == 64) return go(tc_pass1_kernel<64>, Pass1Cfg<64>::kTotal);
  return cudaErrorInvalidValue;
}

cudaError_t launch_tc_pass2(int RP, const Tables& t, const Tile* tiles, int ntiles, const void* maps, Launch l) {
  if (ntiles == 0) return cudaSuccess;
  auto go = [&](auto kernel, size_t smem) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_pdl(kernel, dim3(l.grid), dim3(kTcThreads), smem, l.stream, t, tiles, ntiles, static_cast<const uint8_t*>(maps));
  };
  if (RP == 16) return go(tc_pass2_kernel<16>, Pass2Cfg<16>::kTotal);
  if (RP == 32) return go(tc_pass2_kernel<32>, Pass2Cfg<32>::kTotal);
  if (RP == 64) return go(tc_pass2_kernel<64>, Pass2Cfg<64>::kTotal);
  return cudaErrorInvalidValue;
}

}  // namespace lqsgd


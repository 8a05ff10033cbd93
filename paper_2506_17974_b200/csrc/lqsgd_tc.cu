// Tensor-core passes of the LQ-SGD round for padded rank >= 16 (Blackwell, sm_100a).
//
// At rank 16 and above the products of Algorithm 1 cost more FP32 instructions per byte than the
// CUDA cores can issue at HBM speed.  These kernels run them on tcgen05, with fp32 accumulators
// in tensor memory (TMEM) and every fp32 operand fed as a sum of narrow terms.
//
// Pass 2 (Q_w = M_w^T P_bar, Alg. 1).  One tcgen05.mma with M = 128 costs about 90 cycles
// whatever N <= 128 is (the feed of the A operand bounds it), so the streamed matrix must pass
// through the tensor core once, with as few instructions per byte as possible:
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
constexpr int kTcMStages = 8;         // ring of M pieces (16 KB each)
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
__device__ __forceinline__ void drain(uint64_t* bar, uint32_t parity) {
  for (uint32_t i = 0; i < kWaitLimit && !mbar_try(bar, parity); ++i) {}
}

// Stages a tile takes: its rows in pieces of 32, rounded up to whole operand slots (a piece past
// the layer's last row reads as zeros and costs no memory traffic).
__device__ __forceinline__ int tile_stages(int nrows) {
  return (nrows + kTcSlotK - 1) / kTcSlotK * kTcPair;
}

template <int RP>
struct Pass2Cfg {
  static constexpr int kN = 3 * RP;                                      // stacked bf16 terms of P_bar
  static constexpr int kDStride = kN <= 64 ? 64 : (kN <= 128 ? 128 : 256);   // TMEM columns per accumulator
  static constexpr int kDBufs = (2 * kDStride + kTcAB * kTcSlotK <= 512) ? 2 : 1;
  static constexpr int kACol0 = kDBufs * kDStride;
  static constexpr int kTmemCols = (kACol0 + kTcAB * kTcSlotK) <= 256 ? 256 : 512;
  static constexpr uint32_t kBBytes = kN * 128;                          // one B stage: 3 RP rows of 64 bf16
  static constexpr uint32_t kBStride = (kBBytes + 1023) / 1024 * 1024;   // stages stay 1024-byte aligned
  static constexpr uint32_t kBOff = kTcMStages * kTcMBytes;
  static constexpr uint32_t kBarOff = kBOff + kTcAB * kTcPair * kBStride;
  static constexpr int kBars = 2 * kTcMStages + 2 * kTcAB + 2 + 2 + 1;
  static constexpr uint32_t kTotal = kBarOff + kBars * 8 + 16 + 1024;    // + abort flag, TMEM slot, alignment slack
  static_assert(kACol0 + kTcAB * kTcSlotK <= 512, "tensor memory");
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
  uint64_t* m_full = bars;                       // [kTcMStages] TMA landed
  uint64_t* m_empty = m_full + kTcMStages;       // [kTcMStages] consumer warps have the piece in registers
  uint64_t* ab_full = m_empty + kTcMStages;      // [kTcAB] slot ready: A written to TMEM (4 warps per stage) and B landed
  uint64_t* ab_empty = ab_full + kTcAB;          // [kTcAB] the MMAs that read buffer i have completed
  uint64_t* d_full = ab_empty + kTcAB;           // [2] accumulator complete
  uint64_t* d_empty = d_full + 2;                // [2] accumulator drained
  uint64_t* fin = d_empty + 2;                   // [1] every MMA of this CTA has completed
  volatile int* abort_flag = reinterpret_cast<volatile int*>(fin + 1);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(fin + 1) + 1;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < kTcMStages; ++s) { mbar_init(m_full + s, 1); mbar_init(m_empty + s, 4); }
    for (int s = 0; s < kTcAB; ++s) { mbar_init(ab_full + s, 4 * kTcPair + 1); mbar_init(ab_empty + s, 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(d_full + s, 1); mbar_init(d_empty + s, 4); }
    mbar_init(fin, 1);
    *abort_flag = 0;
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
        const int s = kc % kTcMStages;
        if (!warp_wait(m_empty + s, ((kc / kTcMStages) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        if (lane == 0) {
          mbar_arrive_expect_tx(m_full + s, kTcMBytes);
          tma_load_3d(mring + (size_t)s * (kTcMBytes / 4), map, tl.col0, tl.row0 + k * kTcK, tl.worker, m_full + s);
        }
      }
    }
    if (!ok && lane == 0)
      for (uint32_t it = kc > (uint32_t)kTcMStages ? kc - kTcMStages : 0; it < kc; ++it)
        drain(m_full + it % kTcMStages, (it / kTcMStages) & 1);
  } else if (warp == 1) {
    // ---- B loader: rows [row0 + 32 k, +32) of the stacked P_bar terms
    uint32_t kc = 0;
    bool ok = true;
    for (int ti = blockIdx.x; ti < ntiles && ok; ti += gridDim.x) {
      const Tile tl = tiles[ti];
      const uint8_t* map = maps + ((size_t)tl.layer * kTcMapsPerLayer + 1) * kTcMapBytes;
      const int nslots = tile_stages(tl.nrows) / kTcPair;
      for (int k = 0; k < nslots; ++k, ++kc) {            // kc counts slots here
        const int s = kc % kTcAB;
        if (!warp_wait(ab_empty + s, ((kc / kTcAB) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
        if (lane == 0) {
          mbar_arrive_expect_tx(ab_full + s, kTcPair * S::kBBytes);
#pragma unroll
          for (int h = 0; h < kTcPair; ++h)
            tma_load_2d(bring + (size_t)(s * kTcPair + h) * S::kBStride, map, tl.row0 + (k * kTcPair + h) * kTcK, 0, ab_full + s);
        }
      }
    }
    if (!ok && lane == 0)
      for (uint32_t it = kc > (uint32_t)kTcAB ? kc - kTcAB : 0; it < kc; ++it) drain(ab_full + it % kTcAB, (it / kTcAB) & 1);
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
          const int s = kc % kTcAB;
          if (!thread_wait(ab_full + s, (kc / kTcAB) & 1, abort_flag)) { ok = false; break; }
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
      drain(fin, 0);
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
#pragma unroll
      for (int j0 = 0; j0 < RP; j0 += 16) {
        uint32_t a[16], b[16], c[16];
        tc_ld16(taddr + j0, a);
        tc_ld16(taddr + RP + j0, b);
        tc_ld16(taddr + 2 * RP + j0, c);
        tc_wait_ld();
        if (col < L.m) {
#pragma unroll
          for (int j = 0; j < 16; j += 4) {
            float4 o;
            o.x = (__uint_as_float(c[j]) + __uint_as_float(b[j])) + __uint_as_float(a[j]);
            o.y = (__uint_as_float(c[j + 1]) + __uint_as_float(b[j + 1])) + __uint_as_float(a[j + 1]);
            o.z = (__uint_as_float(c[j + 2]) + __uint_as_float(b[j + 2])) + __uint_as_float(a[j + 2]);
            o.w = (__uint_as_float(c[j + 3]) + __uint_as_float(b[j + 3])) + __uint_as_float(a[j + 3]);
            *reinterpret_cast<float4*>(dst + j0 + j) = o;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(d_empty + db);
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
        const int s = kc % kTcMStages;
        const uint32_t slot = kc / kTcPair, ab = slot % kTcAB;
        if (!warp_wait(m_full + s, (kc / kTcMStages) & 1, abort_flag, lane)) { ok = false; break; }
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
        if (!warp_wait(ab_empty + ab, ((slot / kTcAB) & 1) ^ 1, abort_flag, lane)) { ok = false; break; }
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

// Fills kTcMapsPerLayer tensor maps per layer (host memory, 128 bytes each); layers that the
// tensor-core passes do not take get zeros.
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
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return LQSGD_ERR_CUDA;
    }
    {   // stacked bf16 terms of P_bar^T, [3 RP][nt] words (a bf16 value twice per word): 32 rows of P_bar
      const cuuint64_t dim[2] = {(cuuint64_t)L.nt, (cuuint64_t)(3 * RP)};
      const cuuint64_t stride[1] = {(cuuint64_t)L.nt * 4};
      const cuuint32_t box[2] = {kTcK, (cuuint32_t)(3 * RP)}, es[2] = {1, 1};
      if (encode(&maps[i * kTcMapsPerLayer + 1], CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, L.Pbt, dim, stride, box, es,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return LQSGD_ERR_CUDA;
    }
  }
  return LQSGD_OK;
}

cudaError_t launch_tc_pass2(int RP, const Tables& t, const Tile* tiles, int ntiles, const void* maps, Launch l) {
  if (ntiles == 0) return cudaSuccess;
  if (RP != 16) return cudaErrorInvalidValue;
  using S = Pass2Cfg<16>;
  cudaError_t e = cudaFuncSetAttribute(tc_pass2_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)S::kTotal);
  if (e != cudaSuccess) return e;
  return launch_pdl(tc_pass2_kernel<16>, dim3(l.grid), dim3(kTcThreads), S::kTotal, l.stream, t, tiles, ntiles,
                    static_cast<const uint8_t*>(maps));
}

}  // namespace lqsgd


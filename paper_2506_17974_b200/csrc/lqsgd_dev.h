// Device-side tables shared by the host planner (lqsgd_api.cu) and the kernels
// (lqsgd_kernels.cu).  Internal to the library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace lqsgd {

constexpr int kMaxRank = 64;           // padded rank 64: the tensor-core passes' shared memory and tensor memory end there
constexpr int kPassThreads = 256;      // threads per CTA of the three streaming passes
constexpr int kPass1Rows = 32;         // rows per pass-1 tile: 8 warps x 4 rows
constexpr int kFactorBlockRows = 128;  // rows of P (or Q) per block of the small factor kernels
constexpr int kExchangeChunk = 256;    // factor elements per block of the exchange kernel

// One matrix layer (n x m), as the kernels see it.  Factors are stored with a row stride of
// RP floats (rank padded to 1, 2, 4, 8, 16, 32 or 64); columns >= r are kept zero.
struct LayerDev {
  int32_t n, m, r;            // r = r_eff
  int32_t vec;                // 1: m % 4 == 0, rows are 16-byte aligned -> float4 path
  int32_t ncc;                // column chunks of pass 1 (P partial sums)
  int32_t nrb;                // row chunks of pass 2 (Q partial sums)
  int32_t npb, nqb;           // factor blocks: ceil(n/128), ceil(m/128)
  int32_t user_index;         // index in the caller's layer list
  int32_t mt;                 // row stride of Qt: m rounded up to a multiple of 4
  int32_t tc;                 // 1: the tensor-core passes take this layer (padded rank >= 16, m % 4 == 0)
  int32_t nt;                 // row stride of Pbt: n rounded up to a multiple of 4
  int32_t kcat;               // row stride of Pcat / Qcat: 3 RP rounded up to a multiple of 32
  float* E;                   // [W][n][m]   error buffer; holds M between pass 1 and pass 3
  float* Q;                   // [m][RP]     warm start, becomes Q_bar
  float* Qt;                  // [RP][mt]    transposed copy of Q read by pass 1 and pass 3;
                              // tc layers: [2 RP][mt], rows RP.. hold the tf32 remainders of rows 0..
  float* Pbt;                 // tc layers: [3 RP][nt] words: P_bar transposed, as three stacked bf16 terms (pass 2 operand)
  float* Pcat;                // tc layers: [n][kcat]  P_bar | P_bar | tf32 remainder of P_bar | 0   (pass 3 operand)
  float* Qcat;                // tc layers: [m][kcat]  Q_bar | tf32 remainder of Q_bar | Q_bar | 0
  float* Ppart;               // [W][ncc][n][RP]
  float* Praw;                // [W][n][RP]  (== Ppart when ncc == 1)
  float* P;                   // [W][n][RP]  orthonormal
  float* Pbar;                // [n][RP]
  float* Qpart;               // [W][nrb][m][RP]
  float* Qw;                  // [W][m][RP]  (== Qpart when nrb == 1)
  double* gram_part;          // [W][npb][RP*RP]
  double* chol;               // padded rank >= 32: [W][RP*RP + 2 RP]  Cholesky factor L (row-major), 1 / diag, dropped flags
  float* maxp;                // [W][npb] block maxima of |P|; with column scales [W][npb][RP], one per column
  float* maxq;                // [W][nqb] (or [W][nqb][RP])
  float* scales;              // [2 RP]: s_P at [0], s_Q at [1]; with column scales s_P[j] at [j], s_Q[j] at [RP + j]
  uint64_t pay_scale_off, pay_p_off, pay_q_off;   // byte offsets inside one worker's payload
  // What the steps after a pass add up.  A layer with many partial sums (more than kFoldAbove) has them summed in
  // groups of kFoldGroup first, by many CTAs (fold_kernel); the step then adds the groups' sums, in order.
  const float* Psum;          // [W][nps][n][RP]: Ppart (nps = ncc) or the folded partials
  const float* Qsum;          // [W][nqs][m][RP]: Qpart (nqs = nrb) or the folded partials
  const double* gram_sum;     // [W][ngs][RP*RP]: gram_part (ngs = npb) or the folded block Grams
  int32_t nps, nqs, ngs;
  int32_t qfused;             // 1: the tensor-core pass 2 holds the whole sum Q_w (one row chunk) and takes the block maxima of
                              // |Q_w| itself (its epilogue; p_apply zeroes them first): no q_reduce blocks for this layer
};

constexpr int kFoldAbove = 64;     // partial sums per layer and worker above which they are folded first
constexpr int kFoldGroup = 32;     // partial sums per fold group
constexpr int kFoldElems = 256;    // elements of a plane per CTA of the fold kernel

// One CTA of the fold kernel: dst[e] = src[e] + src[plane + e] + ... (count planes, in order), e0 <= e < e0 + kFoldElems.
struct FoldJob {
  const void* src;            // the group's first plane
  void* dst;
  uint32_t plane;             // elements per plane
  uint32_t e0;
  uint16_t count;             // planes in this group (1..kFoldGroup)
  uint16_t is_double;         // 0: float planes, 1: double planes
  uint32_t pad_;
};

// One 1-D tensor.
struct VectorDev {
  int32_t len;
  int32_t user_index;
  uint64_t pay_off;           // byte offset inside one worker's payload: fp32 values (4-byte aligned) or code stream
  uint64_t pay_scale_off;     // quantised variant: where the tensor's fp32 scale goes (4-byte aligned)
};

// A rectangular piece of one layer handled by one CTA of a streaming pass.
struct Tile {
  int32_t layer;              // index into the LayerDev table
  int32_t worker;             // unused by pass 3 (it loops over the workers)
  int32_t row0, nrows;
  int32_t col0, ncols;
  int32_t part;               // pass 1: column-chunk index; pass 2: row-chunk index
  int32_t pad;                // staged passes: 1 = plain tile (whole rows of a small layer with unaligned rows,
                              // taken by the consumers with ordinary loads), else 0
};

// A block of rows of one worker's factor, handled by one CTA of a small factor kernel.
struct FactorBlock {
  int32_t layer, worker, blk, pad;
};

// A chunk of kExchangeChunk factor elements of one layer, all workers.
struct ExchangeChunk {
  int32_t layer, chunk;
};

struct Tables {
  const LayerDev* layers;
  const float* const* grads;  // [n_mat][W] device pointers, by LayerDev index
  float* const* ghat;         // [n_mat]; an entry may be null: G_hat of that layer is not written
  float* const* weights;      // [n_mat] or null; non-null entry: w <- w - lr * G_hat in pass 3 (Alg. 1 model update)
  float lr;
  uint8_t* payload;           // [W][payload_stride]
  uint64_t payload_stride;
  uint32_t* status;           // [n_mat]
  const uint8_t* gmaps;       // [n_mat][W] tensor maps of the gradients (layers on the tensor-core passes), or null
  int32_t W;
  int32_t col_scales;         // 1: one quantiser scale per factor column (variant), 0: one per factor
  int32_t clear_status;       // > 0 only in the round's first pass-1 launch: that many status words are zeroed by CTA 0
  // Test support (lqsgd_test_expire_wait; all zero in normal operation): the bounded waits of the staged and
  // tensor-core passes give up after wait_limit timed polls instead of the built-in limit, and the loader of
  // CTA 0 of pass test_skip_pass (1, 2 or 3) issues no copies from its stage number test_skip_stage on, so
  // that the waits on those stages run out.  (From that stage ON, not that stage alone: a ring's barrier
  // tells phases apart by parity only, so a waiter one ring turn further would take the missing phase for
  // the one before it.)  Every address stays valid; only waits expire.
  uint32_t wait_limit;
  int32_t test_skip_pass;
  int32_t test_skip_stage;
};
__device__ __forceinline__ bool test_skips_stage(const Tables& t, int pass, uint32_t stage) {
  return t.test_skip_pass == pass && blockIdx.x == 0 && stage >= (uint32_t)t.test_skip_stage;
}

struct QuantTables {
  const float* thr;           // [L-1] ascending decision thresholds on |x|/s
  const float* deq;           // [2*W*(L-1)+1] expand(S / (W (L-1))), index S + W (L-1); with avg_values the
                              // table is the one of a single worker: [2*(L-1)+1], index (+-k) + (L-1)
  int32_t bits;
  int32_t avg_values;         // 1: dequantise every worker's code, then average (variant); 0: Algorithm 1's order
};

// Programmatic dependent launch: every kernel of the round is launched so that its launch may
// overlap the tail of the kernel before it in the stream, and begins with pdl_wait(), which
// returns once that kernel has completed and its writes are visible.
__device__ __forceinline__ void pdl_wait() {
#if defined(__CUDA_ARCH__)
  asm volatile("griddepcontrol.wait;" ::: "memory");
#endif
}
// Called before pdl_wait() by the pass kernels: the CTA's first tile and that tile's layer entry (tables written at
// create, never changed) are asked for while the kernel in front is still finishing, the entry into L2 only, so that
// the loads after the wait find them close by.
__device__ __forceinline__ void prefetch_first_tile(const Tables& t, const Tile* tiles, int ntiles) {
#if defined(__CUDA_ARCH__)
  if (threadIdx.x == 0 && (int)blockIdx.x < ntiles) {
    const int layer = __ldg(&tiles[blockIdx.x].layer);
    const char* e = reinterpret_cast<const char*>(t.layers + layer);
    asm volatile("prefetch.global.L2 [%0];" ::"l"(e));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(e + sizeof(LayerDev) - 1));
  }
#endif
}
// The status words of a round start at zero.  The first pass-1 kernel of the round clears them itself (CTA 0, right
// after its wait on the previous kernel), which saves a memset node between two rounds and lets this kernel's launch
// overlap the previous round's tail.  Nothing can set a bit before the clear: the only bits a pass-1 kernel sets are
// time-outs, and a wait gives up after 2^18 polls (milliseconds), while CTA 0 of a grid that fits the GPU at once
// runs its first instructions in the kernel's first microseconds; every other bit comes from later kernels.
__device__ __forceinline__ void clear_status_words(const Tables& t) {
  if (t.clear_status > 0 && blockIdx.x == 0)
    for (int i = threadIdx.x; i < t.clear_status; i += blockDim.x) t.status[i] = 0u;
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

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

struct Launch {
  cudaStream_t stream;
  int grid;
};

cudaError_t launch_pass1(int RP, const Tables& t, const Tile* tiles, int ntiles, Launch l);
cudaError_t launch_p_reduce_gram(int RP, const Tables& t, const FactorBlock* fb, int nfb, Launch l);
cudaError_t launch_p_apply(int RP, const Tables& t, const FactorBlock* fb, int nfb, Launch l);
// padded rank >= kCholSplitRP: the Cholesky factor of each (layer, worker) once, by a CTA of its own, instead of again in
// every CTA of p_apply (at rank 64 the factorisation is the long part); fb lists one entry per (layer, worker)
constexpr int kCholSplitRP = 32;
cudaError_t launch_p_chol(int RP, const Tables& t, const FactorBlock* fb, int nfb, Launch l);
cudaError_t launch_fold(const FoldJob* jobs, int njobs, Launch l);
// Orthonormalize in one launch for layers of at most kOrthSmallMaxRows rows at RP <= 8: one CTA per (layer, worker)
constexpr int kOrthSmallMaxRows = 512;
cudaError_t launch_p_orth_small(int RP, const Tables& t, const FactorBlock* fb, int nfb, Launch l);
// Split exchange (workers on several GPUs).  pack_only: quantise and pack with the scales in
// `scales` ([2][n_mat], agreed between the ranks) and also write the streams into `send`
// ([which][W][region_bytes], contiguous, ready for an all-gather); no sum, no dequantisation.
struct SplitExchange {
  int32_t pack_only;
  int32_t n_mat;
  int32_t ns;                 // scales per factor and layer: 1, or RP with one scale per column
  const float* scales;        // [2][n_mat][ns]
  uint8_t* send[2];
  uint64_t region_bytes[2];   // bytes of all layers' P (or Q) streams of one worker
  uint64_t region_off[2];     // offset of that region inside a payload
};
// The round's 1-D tensors (fp32 mean over the workers): tables, the step's pointers, what the model update needs.
struct VectorJob {
  const VectorDev* vecs;
  const ExchangeChunk* chunks;   // (tensor, block of 256 entries)
  int32_t nchunks;
  int32_t W_total;               // workers of all ranks (the divisor of the mean)
  const float* const* vgrads;    // [n_vec][W]
  float* const* vghat;           // [n_vec], entries may be null
  float* const* vweights;        // [n_vec] or null
  float lr;
  float* xvec;                   // workers on several GPUs: this rank's shares of the means go here (all tensors, in
                                 // payload order, contiguous) for ONE all-reduce, instead of into vghat / vweights
  uint64_t xvec_base;            // payload offset of the first 1-D tensor's values
};
// ride: the 1-D tensors' blocks appended to this launch (or null)
cudaError_t launch_exchange(int RP, int which /*0 = P, 1 = Q*/, const Tables& t, const QuantTables& q,
                            const ExchangeChunk* ch, int nch, const SplitExchange& sx, const VectorJob* ride, Launch l);
// Guard blocks of the workspace (256 bytes each at base + offs[i]): result == null fills them with the pattern, else
// counts the words that no longer hold it into result[0] and keeps the smallest byte offset of one in result[1].
cudaError_t launch_guards(char* base, const uint64_t* offs, int n, uint32_t pattern, unsigned long long* result, cudaStream_t st);
cudaError_t launch_unpack_codes(const uint8_t* stream, int count, int bits, uint8_t* out, cudaStream_t st);
cudaError_t launch_scale_reduce(int RP, const Tables& t, int which, float* scales, int n_mat, Launch l);
cudaError_t launch_sum_dequant(int RP, int which, const Tables& t, const QuantTables& q, const ExchangeChunk* ch,
                               int nch, const SplitExchange& sx, const uint8_t* gathered, int n_streams, Launch l);
cudaError_t launch_q_transpose(const float* Q, float* Qt, float* Qcat, int m, int RP, int mt, int kcat, int tc,
                               cudaStream_t stream);
cudaError_t launch_pass2(int RP, const Tables& t, const Tile* tiles, int ntiles, Launch l);
cudaError_t launch_q_reduce(int RP, const Tables& t, const FactorBlock* fb, int nfb, Launch l);
cudaError_t launch_pass3(int RP, const Tables& t, const Tile* tiles, int ntiles, Launch l);
// Variant: 1-D tensors log-quantised like a factor (one CTA per tensor).
cudaError_t launch_vectors_quant(const VectorDev* vecs, int nvecs, const float* const* vgrads, float* const* vghat,
                                 float* const* vweights, float lr, uint8_t* payload, uint64_t payload_stride, int W,
                                 const QuantTables& q, Launch l);
cudaError_t launch_vectors(const VectorJob& vj, uint8_t* payload, uint64_t payload_stride, int W, Launch l);
// after the all-reduce of xvec: the means go to vghat, and into the weights (model update)
cudaError_t launch_vectors_finish(const VectorJob& vj, Launch l);
// Bulk-copy staged passes (lqsgd_stream.cu): layers with m % 4 == 0 and RP <= 8.  One CTA per SM,
// 512 consumer threads.  The copy engine limits the number of bulk copies in flight, not their
// bytes, so tiles are wide (few, large row segments per stage) and a tile that spans whole rows
// is fetched with ONE copy per stage (consecutive rows are contiguous).
constexpr int kStreamMaxRP = 8;
constexpr int kStreamConsumers = 512;
constexpr int kStreamPlainElems = 65536;  // largest layer (elements per worker) with unaligned rows the staged kernels take as plain tiles
constexpr int kStreamPlainRows = 16;      // rows of a plain tile: one per consumer warp
constexpr int kStreamSlabFloats = 9216;   // one stage of one array: 36 KB = 16 x 576 = 8 x 1152 = 2 x 4608 floats

// Widest tile (columns) the staged passes take at this padded rank: a thread keeps the Q rows
// of all the column quads it owns in registers (quads per thread x 4 x RP <= 32 floats).
__host__ __device__ inline int stream_max_cols(int RP) { return RP >= 8 ? 2048 : (RP == 4 ? 4096 : 6144); }

// How the 512 consumers cover one stage of a tile `ncols` wide.
struct StreamGeo {
  int quads;   // float4 columns per row
  int qpt;     // quads per thread (1..3); > 1 only when one row needs more than 512 threads
  int tpr;     // threads per row (multiple of 32, <= 512)
  int ng;      // row groups working side by side (512 / tpr)
  int rpg;     // rows per group per stage (<= stream_rows_per_thread(RP))
  int R;       // rows per stage
};
__host__ __device__ inline int stream_rows_per_thread(int RP) { return RP >= 8 ? 4 : 8; }
__host__ __device__ inline StreamGeo stream_geo(int ncols, int RP) {
  StreamGeo g;
  g.quads = ncols >> 2;
  g.qpt = (g.quads + kStreamConsumers - 1) / kStreamConsumers;
  g.tpr = g.quads >= kStreamConsumers ? kStreamConsumers : ((g.quads + 31) & ~31);
  g.ng = kStreamConsumers / g.tpr;
  int R = kStreamSlabFloats / ncols;
  const int cap = g.ng * stream_rows_per_thread(RP);
  if (R > cap) R = cap;
  if (R < 1) R = 1;
  g.R = R;
  g.rpg = (R + g.ng - 1) / g.ng;
  return g;
}
// Tensor-core passes (lqsgd_tc.cu): layers with m % 4 == 0 at padded rank >= 16.  The products run
// on tcgen05 with every fp32 operand fed as a sum of narrow terms, fp32 accumulation in tensor
// memory.  `maps` is the layer-major array of tensor maps (kTcMapsPerLayer per layer) that
// tc_encode_maps() filled.
constexpr int kTcMapsPerLayer = 6;   // 0: M as [W][n][m], box 128 x 32 x 1;  1: Pbt, box 32 x 3RP, 128-byte swizzle;
                                     // 2: E / M as [W][n][m], box 32 x 128 x 1, swizzled;  3: Qt, box 32 x 2RP, swizzled
                                     // 4: Pcat, 5: Qcat, box 32 x 128, swizzled
constexpr int kTcRowsPerTile = 128;  // rows of a pass-1 tile: the M extent of one MMA
constexpr int kTcPass1Cols = 1152;   // most columns of a pass-1 tile (multiple of 32): small enough to balance the SMs
constexpr int kTcMapBytes = 128;
constexpr int kTcRowChunk = 4096;    // most rows of a layer one pass-2 tile sums over (multiple of 64)
int tc_encode_maps(const LayerDev* host_layers, int n_layers, int W, int RP, void* host_maps_out);   // 0 or LQSGD_ERR_CUDA
// one map per (layer, worker) over the caller's gradients (grads: [n_layers][W] device pointers); out: [n_layers][W] maps
int tc_encode_grad_maps(const LayerDev* host_layers, int n_layers, int W, const void* const* grads, void* host_maps_out);
cudaError_t launch_tc_pass2(int RP, const Tables& t, const Tile* tiles, int ntiles, const void* maps, Launch l);
// passes 1 and 3 hand their tiles out at run time, in list order: sched = {draw counter, CTAs that have left}, zero before
// the first launch (the kernels leave it zero); l.grid CTAs
cudaError_t launch_tc_pass1(int RP, const Tables& t, const Tile* tiles, int ntiles, int* sched, const void* maps,
                            Launch l);
cudaError_t launch_tc_pass3(int RP, const Tables& t, const Tile* tiles, int ntiles, int* sched, const void* maps,
                            Launch l);
// One-launch round (lqsgd_resident.cu) for sets whose M fits in the SMs' shared memory: one cooperative grid,
// one CTA of kResThreads threads per SM, tiles of M resident from pass 1 to pass 3, grid barriers between the steps.
constexpr int kResThreads = 512;
constexpr int kResMaxTiles = 16;       // tiles one CTA may hold (one shared-memory barrier each)
constexpr int kResMaxTileRows = 256;   // rows of a tile (its rows of P_bar wait in scratch)
constexpr int kResMaxTileCols = 1024;  // columns of a tile (its rows of Q_bar wait in scratch)
constexpr int kResBarriers = 6;        // grid barriers per launch at most (counters per set)
constexpr int kResStamps = 12;         // timeline stamps per launch (then one word holding their number)
struct ResTile {
  int32_t layer, worker;
  int32_t row0, nrows, col0, ncols;
  int32_t part_c, part_r;     // column chunk (partial sums of P), row chunk (partial sums of Q)
  int32_t smem_off;           // floats from the start of the CTA's resident area (multiple of 4)
  int32_t plain;              // 1: the layer's rows are not 16-byte aligned: whole rows, ordinary loads and stores
  int32_t writes_ghat;        // 1: this tile (worker 0's) also writes G_hat and applies the model update
  int32_t pad;
};
struct ResidentArgs {
  const ResTile* tiles;
  const int* cta_begin;       // [grid + 1]: CTA b holds tiles [cta_begin[b], cta_begin[b + 1])
  const FactorBlock* fbS; int32_t nfbS;
  const FactorBlock* fbP; int32_t nfbP;
  const FactorBlock* fbQ; int32_t nfbQ;
  const ExchangeChunk* chP; int32_t nchP;
  const ExchangeChunk* chQ; int32_t nchQ;
  QuantTables qp, qq;
  VectorJob vj;               // nchunks == 0: no 1-D tensors
  uint32_t* sync;             // [1 + 2 * kResBarriers]: launch counter, two sets of barrier counters
  uint64_t* stamps;           // [kResStamps + 1]: CTA 0's timeline of the launch in ns, then the number of stamps
};
size_t resident_scratch_bytes(int RP);   // shared memory per CTA that is not available to tiles
cudaError_t launch_resident(int RP, const Tables& t, const ResidentArgs& a, int grid, size_t smem_bytes, cudaStream_t stream);
cudaError_t resident_max_grid(int RP, size_t smem_bytes, int sm_count, int* grid_out);   // 0: the kernel does not fit
cudaError_t launch_stream_pass1(int RP, const Tables& t, const Tile* tiles, int ntiles, Launch l);
cudaError_t launch_stream_pass3(int RP, const Tables& t, const Tile* tiles, int ntiles, Launch l);
// Resident CTAs per SM of each streaming pass for this RP (for persistent grid sizing).
cudaError_t pass_occupancy(int RP, int* occ1, int* occ2, int* occ3);

}  // namespace lqsgd

// Host side of the LQ-SGD library: argument checking, workspace carving, the tile planner,
// table upload and the per-step launch sequence behind the C ABI of include/lqsgd.h.
#include "../../include/lqsgd.h"
#include "lqsgd_dev.h"
#include "lqsgd_stats.h"

#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <array>
#include <cmath>
#include <cstring>
#include <map>
#include <new>
#include <queue>
#include <string>
#include <tuple>
#include <vector>

using namespace lqsgd;

namespace {

thread_local std::string g_cuda_error;

int cuda_fail(cudaError_t e, const char* what) {
  g_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
  return LQSGD_ERR_CUDA;
}
#define CK(call)                                              \
  do {                                                        \
    cudaError_t e__ = (call);                                 \
    if (e__ != cudaSuccess) return cuda_fail(e__, #call);     \
  } while (0)

}  // namespace
namespace lqsgd {
// for the library's other translation units: records the text lqsgd_last_cuda_error() returns
int record_cuda_failure(cudaError_t e, const char* what) { return cuda_fail(e, what); }
}  // namespace lqsgd
namespace {

// NVTX range around the launches of one phase of the round: shows in a timeline tool next to the kernels, costs
// nothing when no tool is attached (the NVTX header only forwards to an injected library).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Hands out 256-byte aligned pieces of the workspace; with base == nullptr it only counts.
// With `guards` set (LQSGD_FLAG_GUARD_WORDS) every piece is followed by kGuardBytes of a fixed pattern that no
// kernel may touch; their offsets are collected for lqsgd_check_guards.
constexpr size_t kGuardBytes = 256;
constexpr uint32_t kGuardPattern = 0xA5C3F00Du;
struct Arena {
  char* base;
  size_t off = 0;
  std::vector<uint64_t>* guards = nullptr;
  explicit Arena(void* b) : base(static_cast<char*>(b)) {}
  template <typename T>
  T* take(size_t count) {
    off = align_up(off, 256);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    if (guards) {
      off = align_up(off, 256);
      guards->push_back(off);
      off += kGuardBytes;
    }
    return p;
  }
};

// Device copies of the tensor-pointer tables of the last kPtrSets distinct pointer sets a context was stepped with: a
// trainer that rotates a few gradient buffers (or always passes the same ones) uploads each table once, and a round
// is then kernels only, with no copy node between two rounds.
constexpr int kPtrSets = 16;

struct MatHost {
  int n, m, r, user_index;
};

struct Plan {
  int RP = 0, W = 0, W_total = 0;             // W_total: workers of all ranks (== W on one GPU)
  std::vector<MatHost> mats;
  std::vector<LayerDev> layers;
  std::vector<VectorDev> vecs;
  std::vector<Tile> tiles1, tiles2, tiles3;      // register-path passes
  std::vector<Tile> stiles1, stiles3;            // bulk-copy staged passes 1 and 3
  std::vector<Tile> tctiles2;                    // tensor-core pass 2
  std::vector<Tile> tctiles1;                    // tensor-core pass 1, handed out at run time in this order
  std::vector<Tile> tctiles3;                    // tensor-core pass 3 (a range of workers per entry), handed out at run time
  int tc_grid = 0;
  std::vector<uint64_t> guards;                  // byte offsets of the guard blocks (LQSGD_FLAG_GUARD_WORDS)
  uint64_t* d_guards = nullptr;
  unsigned long long* d_guard_result = nullptr;  // [2]: words found changed, offset of the first of them
  bool resident = false;                         // the one-launch round takes this set (lqsgd_resident.cu)
  std::vector<ResTile> rtiles;                   // its tiles, grouped by CTA
  std::vector<int> rbegin;                       // [res_grid + 1]
  int res_grid = 0;
  size_t res_smem = 0;                           // dynamic shared memory per CTA
  ResTile* d_rtiles = nullptr;
  int* d_rbegin = nullptr;
  uint32_t* d_rsync = nullptr;                   // launch counter + two sets of grid-barrier counters
  int* d_tcsched = nullptr;                      // tensor-core passes that hand out their tiles at run time
  uint64_t* d_rstamps = nullptr;                 // timeline of the last one-launch round
  std::vector<uint8_t> tcmaps;                   // tensor maps of the tensor-core passes (filled at create)
  std::vector<FactorBlock> fbP, fbQ;             // 128-row blocks of P (layers orthonormalised in two launches) and of Q
  std::vector<FactorBlock> fbS;                  // (layer, worker) of the layers orthonormalised by one CTA
  std::vector<FactorBlock> fbC;                  // padded rank >= 32: (layer, worker) whose Cholesky factor a CTA of its own computes
  FactorBlock* d_fbC = nullptr;
  std::vector<FoldJob> foldP, foldG, foldQ;      // layers with many partial sums: groups summed first (after pass 1, the block Grams, after pass 2)
  FoldJob *d_foldP = nullptr, *d_foldG = nullptr, *d_foldQ = nullptr;
  std::vector<ExchangeChunk> chP, chQ, chV;
  std::vector<float> thrP, thrQ, deqP, deqQ;
  std::vector<lqsgd_layer_layout> layout;     // by user layer index
  size_t payload_bytes = 0, payload_stride = 0;
  size_t elems_total = 0;                     // all layers, one worker
  std::vector<size_t> elem_off;               // by user index, offset in a worker's staging plane
  // device addresses (null when only counting)
  LayerDev* d_layers = nullptr;
  VectorDev* d_vecs = nullptr;
  Tile *d_tiles1 = nullptr, *d_tiles2 = nullptr, *d_tiles3 = nullptr;
  Tile *d_stiles1 = nullptr, *d_stiles3 = nullptr;
  Tile* d_tctiles2 = nullptr;
  Tile* d_tctiles1 = nullptr;
  Tile* d_tctiles3 = nullptr;
  uint8_t* d_tcmaps = nullptr;
  FactorBlock *d_fbP = nullptr, *d_fbQ = nullptr, *d_fbS = nullptr;
  ExchangeChunk *d_chP = nullptr, *d_chQ = nullptr, *d_chV = nullptr;
  float *d_thrP = nullptr, *d_thrQ = nullptr, *d_deqP = nullptr, *d_deqQ = nullptr;
  void** d_ptrs = nullptr;                    // kPtrSets pointer tables, see prepare_step for the layout of one
  uint32_t* d_status = nullptr;
  unsigned long long* d_stats = nullptr;      // [4]: result words of lqsgd_step_stats (one layer at a time)
  uint8_t* d_payload = nullptr;
  float* d_xscales = nullptr;                 // [2][n_mat][ns] scales the ranks agree on (split exchange); ns = 1, or RP per column
  int xscale_ns = 1;
  float* d_xvec = nullptr;                    // the 1-D tensors' means, all in one buffer (split round: one all-reduce)
  size_t vec_elems = 0;
  uint64_t vec_pay_base = 0;                  // payload offset of the first 1-D tensor's values
  uint8_t* d_xsend[2] = {nullptr, nullptr};   // [W][region_bytes]: local P / Q streams, contiguous, for the all-gather
  uint64_t region_off[2] = {0, 0}, region_bytes[2] = {0, 0};
  size_t zero_elems = 0;
  float* d_zero = nullptr;                    // power_iters > 1: zeros, as large as the largest matrix
  void** d_zero_ptrs = nullptr;               // [n_mat * W] pointers to d_zero: the "gradient" of a repeated power step
  uint8_t* d_gmaps = nullptr;                 // tensor-core passes: [kPtrSets][n_mat * W] tensor maps of the gradients, beside the pointer tables
  uint8_t* d_zero_gmaps = nullptr;            // [n_mat * W] the same over d_zero
  bool any_tc = false;
  float* d_stage_g = nullptr;                 // [W][elems_total]
  float* d_stage_ghat = nullptr;              // [elems_total]
  size_t state_begin = 0, state_end = 0;      // byte range to zero at create (E, factors, codes ...)
  size_t bytes = 0;
};

int padded_rank(int r) { return r <= 1 ? 1 : r <= 2 ? 2 : r <= 4 ? 4 : r <= 8 ? 8 : r <= 16 ? 16 : r <= 32 ? 32 : 64; }

int check_config(const lqsgd_shape* shapes, int32_t n_layers, const lqsgd_config* c) {
  if (!shapes || !c || n_layers < 1) return LQSGD_ERR_INVALID_ARG;
  if (c->struct_size != sizeof(lqsgd_config)) return LQSGD_ERR_INVALID_ARG;
  if (c->rank < 1 || c->rank > kMaxRank) return LQSGD_ERR_INVALID_ARG;
  auto bits_ok = [](int b) { return (b >= 2 && b <= 8) || b == 32; };
  if (!bits_ok(c->bits_p) || !bits_ok(c->bits_q)) return LQSGD_ERR_INVALID_ARG;
  if (!(c->alpha > 0.f) || !std::isfinite(c->alpha)) return LQSGD_ERR_INVALID_ARG;
  if (c->workers < 1 || c->workers > 256) return LQSGD_ERR_INVALID_ARG;
  if (c->power_iters < 0 || c->power_iters > 8) return LQSGD_ERR_INVALID_ARG;
  if (c->power_iters > 1 && c->world_workers > c->workers) return LQSGD_ERR_INVALID_ARG;
  if (c->world_workers != 0) {     // workers of all ranks: a multiple of the local ones
    if (c->world_workers < c->workers || c->world_workers > 4096 || c->world_workers % c->workers) return LQSGD_ERR_INVALID_ARG;
  }
  if (c->flags & ~(LQSGD_FLAG_HOST_STAGING | LQSGD_FLAG_REGISTER_PATH | LQSGD_FLAG_AVERAGE_VALUES |
                   LQSGD_FLAG_QUANTIZE_VECTORS | LQSGD_FLAG_COLUMN_SCALES | LQSGD_FLAG_ONE_LAUNCH | LQSGD_FLAG_GUARD_WORDS))
    return LQSGD_ERR_INVALID_ARG;
  for (int i = 0; i < n_layers; ++i) {
    if (shapes[i].rows < 1 || shapes[i].cols < 1) return LQSGD_ERR_BAD_SHAPE;
    if ((int64_t)shapes[i].rows * shapes[i].cols > (int64_t)1 << 30) return LQSGD_ERR_BAD_SHAPE;
  }
  return LQSGD_OK;
}

// Decision thresholds and dequantisation table of the b-bit quantiser (Eq. 4 / Eq. 5):
// boundary between levels k and k+1 at |x|/s = ((1+alpha)^((k+1/2)/(L-1)) - 1)/alpha, stored as
// the smallest fp32 >= that value; deq[S + W(L-1)] = sign(S) ((1+alpha)^(|S|/(W(L-1))) - 1)/alpha.
void quant_tables(int bits, double alpha, int W, std::vector<float>& thr, std::vector<float>& deq) {
  if (bits == 32) { thr.assign(1, 0.f); deq.assign(1, 0.f); return; }   // quantiser bypassed: no tables
  const int L = 1 << (bits - 1);
  const double la = std::log1p(alpha);
  thr.resize(L - 1);
  for (int k = 0; k < L - 1; ++k) {
    const double T = std::expm1((k + 0.5) / (L - 1) * la) / alpha;
    float f = (float)T;
    if ((double)f < T) f = std::nextafterf(f, INFINITY);
    thr[k] = f;
  }
  const int C = W * (L - 1);
  deq.resize(2 * (size_t)C + 1);
  for (int S = -C; S <= C; ++S) {
    const double q = std::fabs((double)S) / C;
    const double x = std::expm1(q * la) / alpha;
    deq[S + C] = (float)(S < 0 ? -x : x);
  }
}

// Picks the largest candidate size whose tile count reaches `want`, else the smallest.
template <typename F>
int pick_size(const std::vector<int>& candidates, size_t want, F count_tiles) {
  for (int c : candidates)
    if (count_tiles(c) >= want) return c;
  return candidates.back();
}

// Finishing time of a list of tile costs handed, in order, to `slots` CTA slots as they become free
// (what the hardware does with a one-CTA-per-tile grid).
double makespan_dynamic(const std::vector<double>& cost, size_t slots) {
  std::priority_queue<double, std::vector<double>, std::greater<double>> free_at;
  for (size_t i = 0; i < std::min(slots, cost.size()); ++i) free_at.push(0.0);
  double end = 0.0;
  for (double c : cost) {
    const double t = free_at.top() + c;
    free_at.pop();
    free_at.push(t);
    end = std::max(end, t);
  }
  return end;
}
// Finishing time when CTA b of `ctas` takes tiles b, b + ctas, ... (the persistent staged kernels).
double makespan_strided(const std::vector<double>& cost, size_t ctas) {
  ctas = std::max<size_t>(1, std::min(ctas, cost.size()));
  std::vector<double> load(ctas, 0.0);
  for (size_t i = 0; i < cost.size(); ++i) load[i % ctas] += cost[i];
  return cost.empty() ? 0.0 : *std::max_element(load.begin(), load.end());
}

// Shared memory one CTA may ask for on this architecture (227 KB).
constexpr size_t kMaxSmemPerCta = 227 * 1024;

// Plan of the one-launch round (lqsgd_resident.cu): cuts every (layer, worker) into tiles that stay in shared
// memory from pass 1 to pass 3 and deals them to one CTA per SM.  Returns false when the set does not qualify:
// too large for the SMs' shared memory together, or a configuration the one-launch kernel does not take.
// On success fills p.rtiles / p.rbegin / p.res_grid / p.res_smem and ncc[li], nrb[li] (chunks of the partial sums).
bool plan_resident(const lqsgd_config& cfg, int sm_count, Plan& p, std::vector<int>& ncc, std::vector<int>& nrb) {
  const int W = p.W, RP = p.RP;
  if (!(cfg.flags & LQSGD_FLAG_ONE_LAUNCH) || (cfg.flags & LQSGD_FLAG_REGISTER_PATH)) return false;
  if ((cfg.flags & LQSGD_FLAG_QUANTIZE_VECTORS) && cfg.bits_p != 32) return false;
  if (RP > 8 || p.W_total != W || cfg.power_iters > 1 || p.mats.empty() || sm_count < 8) return false;
  const size_t fixed = resident_scratch_bytes(RP);
  if (fixed == 0 || fixed + 16384 > kMaxSmemPerCta) return false;
  const size_t cap = (kMaxSmemPerCta - fixed) / 4 / 4 * 4;            // floats of tiles per CTA
  size_t F = 0, rows_total = 0;
  for (auto& mt : p.mats) {
    if (mt.m % 4 != 0 && (size_t)mt.n * mt.m > (size_t)kStreamPlainElems) return false;
    if (mt.m % 4 != 0 && mt.m > kResMaxTileCols) return false;
    F += (size_t)W * mt.n * mt.m;
    rows_total += (size_t)W * mt.n;
  }
  if ((double)F > 0.96 * (double)cap * sm_count) return false;
  // the steps between the passes are spread over the CTAs in blocks of 128 rows or 256 elements: a set with very
  // tall factors would make them, not the passes, the long part
  if (rows_total * RP > (size_t)1 << 20) return false;
  const double fill = (double)F / ((double)cap * sm_count);
  // Tile size: one tile per CTA of the large layers when the set leaves some room (fewest partial sums, one long
  // stream per CTA); a set that nearly fills the shared memory is cut finer so that the tiles pack.  A layer much
  // smaller than a tile stays whole.  Tiles are as wide as a row copy should be (up to kResMaxTileCols columns).
  const int per_cta = fill <= 0.88 ? 1 : 8;
  double T = std::max(8192.0, (double)F / ((double)sm_count * per_cta));
  std::vector<ResTile> tiles;
  for (int attempt = 0; attempt < 60; ++attempt, T *= 1.03) {
    tiles.clear();
    size_t big_tiles = 0;
    for (size_t li = 0; li < p.mats.size(); ++li) {
      const MatHost& mt = p.mats[li];
      const bool plain = mt.m % 4 != 0;
      int cols = mt.m, nc = 1;
      if (!plain && mt.m > kResMaxTileCols) {
        nc = ceil_div(mt.m, kResMaxTileCols);
        cols = (int)align_up((size_t)ceil_div(mt.m, nc), 4);
        nc = ceil_div(mt.m, cols);
      }
      int rows = (int)std::min<double>(kResMaxTileRows, std::max(1.0, std::floor(T / cols)));
      rows = std::min(rows, mt.n);
      const int nr = ceil_div(mt.n, rows);
      rows = ceil_div(mt.n, nr);
      ncc[li] = nc;
      nrb[li] = nr;
      if ((double)rows * cols > 0.5 * T) big_tiles += (size_t)W * nr * nc;
      for (int w = 0; w < W; ++w)
        for (int rb = 0; rb < nr; ++rb)
          for (int cc = 0; cc < nc; ++cc) {
            ResTile tl{};
            tl.layer = (int)li; tl.worker = w;
            tl.row0 = rb * rows; tl.nrows = std::min(rows, mt.n - rb * rows);
            tl.col0 = cc * cols; tl.ncols = std::min(cols, mt.m - cc * cols);
            tl.part_c = cc; tl.part_r = rb;
            tl.plain = plain ? 1 : 0;
            tl.writes_ghat = (w == 0) ? 1 : 0;
            tiles.push_back(tl);
          }
    }
    // one tile per CTA: the large tiles must not need a second round of CTAs
    if (per_cta > 1 || big_tiles <= (size_t)sm_count || T > (double)cap) break;
  }
  // longest tile first to the CTA with the least so far
  std::vector<int> order(tiles.size());
  for (size_t i = 0; i < order.size(); ++i) order[i] = (int)i;
  auto fl = [&](const ResTile& tl) { return align_up((size_t)tl.nrows * tl.ncols, 4); };
  std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return fl(tiles[x]) > fl(tiles[y]); });
  std::vector<std::vector<int>> per(sm_count);
  std::vector<size_t> load(sm_count, 0);
  for (int i : order) {
    int best = -1;
    for (int b = 0; b < sm_count; ++b)
      if ((int)per[b].size() < kResMaxTiles && load[b] + fl(tiles[i]) <= cap && (best < 0 || load[b] < load[best])) best = b;
    if (best < 0) return false;
    per[best].push_back(i);
    load[best] += fl(tiles[i]);
  }
  p.rtiles.clear();
  p.rbegin.assign(sm_count + 1, 0);
  size_t most = 0;
  for (int b = 0; b < sm_count; ++b) {
    size_t off = 0;
    for (int i : per[b]) {
      ResTile tl = tiles[i];
      tl.smem_off = (int)off;
      off += fl(tl);
      p.rtiles.push_back(tl);
    }
    most = std::max(most, off);
    p.rbegin[b + 1] = (int)p.rtiles.size();
  }
  p.res_grid = sm_count;
  p.res_smem = fixed + most * 4;
  return true;
}

// Lays out the workspace and builds every table.  base == nullptr: size only.
void make_plan(const lqsgd_shape* shapes, int n_layers, const lqsgd_config& cfg, void* base, int sm_count,
               Plan& p, bool allow_resident = true) {
  const int W = cfg.workers, RP = padded_rank(cfg.rank);
  p.RP = RP;
  p.W = W;
  p.W_total = cfg.world_workers > 0 ? cfg.world_workers : W;
  p.layout.assign(n_layers, lqsgd_layer_layout{});
  p.elem_off.resize(n_layers);
  for (int i = 0; i < n_layers; ++i) {
    p.elem_off[i] = p.elems_total;
    p.elems_total += align_up((size_t)shapes[i].rows * shapes[i].cols, 4);   // keeps 16-byte alignment
    if (shapes[i].rows > 1 && shapes[i].cols > 1) {
      const int r = std::min({cfg.rank, shapes[i].rows, shapes[i].cols});
      p.mats.push_back({shapes[i].rows, shapes[i].cols, r, i});
    } else {
      p.vecs.push_back({shapes[i].rows * shapes[i].cols, i, 0, 0});
    }
  }
  // ---- payload layout: [scales][1-D fp32][P streams][Q streams]
  size_t off = 0;
  const bool colscales = (cfg.flags & LQSGD_FLAG_COLUMN_SCALES) != 0;   // s_P[r] then s_Q[r] instead of s_P, s_Q
  for (auto& mt : p.mats) { p.layout[mt.user_index].scale_offset = off; off += colscales ? 8 * (size_t)mt.r : 8; }
  const bool qvec = (cfg.flags & LQSGD_FLAG_QUANTIZE_VECTORS) && cfg.bits_p != 32;
  if (qvec)
    for (auto& v : p.vecs) { v.pay_scale_off = off; p.layout[v.user_index].scale_offset = off; off += 4; }
  for (auto& v : p.vecs) {
    v.pay_off = off;
    auto& lo = p.layout[v.user_index];
    lo.vec_offset = off; lo.vec_bytes = qvec ? ((size_t)v.len * cfg.bits_p + 7) / 8 : 4 * (size_t)v.len;
    off += lo.vec_bytes;
  }
  for (auto& mt : p.mats) {
    auto& lo = p.layout[mt.user_index];
    lo.is_matrix = 1; lo.rank_eff = mt.r;
    lo.p_offset = off; lo.p_bytes = ((size_t)mt.n * mt.r * cfg.bits_p + 7) / 8; off += lo.p_bytes;   // bits 32: the fp32 factor
  }
  for (auto& mt : p.mats) {
    auto& lo = p.layout[mt.user_index];
    lo.q_offset = off; lo.q_bytes = ((size_t)mt.m * mt.r * cfg.bits_q + 7) / 8; off += lo.q_bytes;
  }
  p.payload_bytes = off;
  if (!p.mats.empty()) {
    const auto& first = p.layout[p.mats.front().user_index];
    const auto& last = p.layout[p.mats.back().user_index];
    p.region_off[0] = first.p_offset; p.region_bytes[0] = last.p_offset + last.p_bytes - first.p_offset;
    p.region_off[1] = first.q_offset; p.region_bytes[1] = last.q_offset + last.q_bytes - first.q_offset;
  }
  p.payload_stride = align_up(off, 16);

  // ---- a set small enough for the SMs' shared memory runs as one launch; its tiles decide the chunking below
  std::vector<int> res_ncc(p.mats.size(), 1), res_nrb(p.mats.size(), 1);
  p.resident = allow_resident && plan_resident(cfg, sm_count, p, res_ncc, res_nrb);

  // ---- tile sizes
  const size_t slots = (size_t)sm_count * 2, want = 3 * slots;
  // above padded rank 16 the register kernels run scalar only (they keep what the tensor-core passes cannot take)
  auto vec_of = [&](int m) { return (RP <= 16 && m % 4 == 0) ? 4 : 1; };
  auto chunk_width = [&](int m, int cmax) {          // balanced column chunks, multiple of 32*VEC
    const int v = vec_of(m), q = 32 * v;
    const int lim = (v == 4) ? cmax : std::max(q, cmax / 4);
    const int ncc = ceil_div(m, lim);
    return (int)align_up((size_t)ceil_div(m, ncc), q);
  };
  const int c1 = pick_size({2048, 1024, 512}, want, [&](int c) {
    size_t t = 0;
    for (auto& mt : p.mats) t += (size_t)p.W_total * ceil_div(mt.n, kPass1Rows) * ceil_div(mt.m, chunk_width(mt.m, c));
    return t;
  });
  const int r2max = std::max(128, 32 * RP);
  auto colchunks = [&](int m) { return ceil_div(m, 128 * vec_of(m)); };
  auto balanced_rows = [](int n, int rmax) { return ceil_div(n, ceil_div(n, rmax)); };
  // Pass 2 (register kernel, one CTA per tile): rows per tile by a model of the schedule.  A tile costs
  // its rows plus a fixed part (start-up, the sum over the row groups) plus its partial sums' way to
  // memory and back (RP floats per column twice, against one float per column and row); the tiles run
  // in launch order on 0.6 of the CTAs that fit the GPU at once (the pass is bound by bandwidth: beyond
  // that many, more CTAs side by side do not finish sooner), and the longest chain of partial sums that
  // the reduction after the pass adds up costs 0.7 of a row each.  Fewer, larger tiles save partial
  // sums; the model stops where waves would run too empty.  (Fitted to rounds timed over tile sizes.)  The chunking of a sum decides its
  // rounding, so the sizes that set it (here and c1 above) count the workers of ALL ranks: a rank that
  // holds some of the workers then rounds like one process that holds them all.
  const size_t slots2 = (size_t)sm_count * (RP <= 2 ? 4 : (RP <= 8 ? 3 : 1));
  int r2 = r2max;
  {
    double best = -1.0;
    for (int r = r2max; r >= 16; r -= 16) {
      std::vector<double> cost;
      int chain = 0;
      for (auto& mt : p.mats) {
        if (!(cfg.flags & LQSGD_FLAG_REGISTER_PATH) && RP >= 16 && mt.m % 4 == 0) continue;   // tensor-core pass 2
        const int tr = balanced_rows(mt.n, r), nrb = ceil_div(mt.n, tr);
        chain = std::max(chain, nrb);
        for (size_t i = 0; i < (size_t)p.W_total * nrb * colchunks(mt.m); ++i) cost.push_back(tr + 2.0 * RP + 16.0);
      }
      const double t = makespan_dynamic(cost, std::max<size_t>(1, slots2 * 6 / 10)) + 0.7 * chain;
      if (best < 0.0 || t < best * 0.97) { best = t; r2 = r; }     // a smaller size must earn 3 %
    }
  }
  const int r3max = std::max(8, 64 / W);
  const int r3 = pick_size({r3max, std::max(8, r3max / 2), 8}, want, [&](int r) {
    size_t t = 0;
    for (auto& mt : p.mats) t += (size_t)ceil_div(mt.n, balanced_rows(mt.n, r)) * colchunks(mt.m);
    return t;
  });
  // Bulk-copy staged passes: layers with 16-byte aligned rows, RP <= 8.  A layer no wider than
  // stream_max_cols(RP) is one column chunk (its rows are then contiguous: one copy per stage);
  // wider layers get chunks balanced in units of 128 columns.  Row chunks hold a target number
  // of elements and are multiples of the rows one stage takes.
  auto staged = [&](const MatHost& mt) {
    return !p.resident && !(cfg.flags & LQSGD_FLAG_REGISTER_PATH) && RP <= kStreamMaxRP && mt.m % 4 == 0;
  };
  // A small layer with unaligned rows rides in the staged kernels as plain tiles (no launch of its own).
  auto plain = [&](const MatHost& mt) {
    return !p.resident && !(cfg.flags & LQSGD_FLAG_REGISTER_PATH) && RP <= kStreamMaxRP && mt.m % 4 != 0 &&
           (size_t)mt.n * mt.m <= (size_t)kStreamPlainElems;
  };
  // Tensor-core passes: padded rank 16, rows 16-byte aligned.
  auto on_tc = [&](const MatHost& mt) {
    return !(cfg.flags & LQSGD_FLAG_REGISTER_PATH) && RP >= 16 && mt.m % 4 == 0;
  };
  auto staged_cols = [&](int m) {                      // list of (col0, ncols)
    std::vector<std::pair<int, int>> out;
    const int maxc = stream_max_cols(RP);
    if (m <= maxc) { out.push_back({0, m}); return out; }
    const int units = ceil_div(m, 128), ncc = ceil_div(units, maxc / 128);
    int u0 = 0;
    for (int c = 0; c < ncc; ++c) {
      const int nu = units / ncc + (c < units % ncc ? 1 : 0);
      out.push_back({u0 * 128, std::min(nu * 128, m - u0 * 128)});
      u0 += nu;
    }
    return out;
  };
  auto stage_rows = [&](int m) {                        // most rows a stage of this layer takes
    int r = 1;
    for (auto& c : staged_cols(m)) r = std::max(r, stream_geo(c.second, RP).R);
    return r;
  };
  auto widest = [&](int m) {
    int w = 0;
    for (auto& c : staged_cols(m)) w = std::max(w, c.second);
    return w;
  };
  // rows per tile: about `elems` elements, at least rmin rows, balanced over n, multiple of R
  auto tile_rows = [&](int n, int m, size_t elems, int rmin) {
    const int R = stage_rows(m);
    int r = (int)std::max<size_t>(elems / (size_t)widest(m), (size_t)std::max(rmin, R));
    r = std::min(r, n);
    r = ceil_div(n, ceil_div(n, r));
    return (int)align_up((size_t)r, R);
  };
  // Tile sizes of the staged passes, again by a model of the schedule: CTA b of one per SM takes tiles
  // b, b + SMs, ... in table order.  A tile costs its bytes (in full 36 KB stages; pass 3: every
  // worker's, plus G_hat once), a little per stage (barriers) and a fixed start (its rows of Q).
  // Small tiles balance the SMs, large ones save starts.  The two constants were fitted to measured
  // pass times over tile sizes on the ResNet-18 set and on single matrices of 16 to 200 M elements;
  // pass 1 then ran fastest at the model's minimum, pass 3 at the smallest size within 1 % of it.
  constexpr double kStageCost = 0.05, kTileCost = 0.1;
  auto staged_makespan = [&](size_t elems, bool pass3) {
    std::vector<double> cost;
    for (auto& mt : p.mats) {
      if (!staged(mt)) continue;
      const auto scols = staged_cols(mt.m);
      const int tr = tile_rows(mt.n, mt.m, elems, 1);
      for (int rb = 0; rb < ceil_div(mt.n, tr); ++rb)
        for (auto& c : scols) {
          const int nrows = std::min(tr, mt.n - rb * tr);
          const double full = (double)nrows * c.second / kStreamSlabFloats;
          const double nst = ceil_div(nrows, stream_geo(c.second, RP).R);
          if (pass3) cost.push_back(W * (full + kStageCost * nst) + 0.5 * full + kTileCost);
          else for (int w = 0; w < W; ++w) cost.push_back(full + kStageCost * nst + kTileCost);
        }
    }
    return makespan_strided(cost, (size_t)sm_count);
  };
  auto pick_staged = [&](bool pass3) {
    size_t best_e = 0;
    double best = -1.0;
    for (int i = 2; i <= 32; ++i) {
      const int k = pass3 ? i : 34 - i;            // pass 3 from the smallest size up, pass 1 from the largest down
      const size_t e = pass3 ? std::max<size_t>(1, (size_t)4096 * k / W) : (size_t)4096 * k;
      const double t = staged_makespan(e, pass3);
      if (best < 0.0 || t < best * (pass3 ? 0.99 : 0.995)) { best = t; best_e = e; }
    }
    return best_e;
  };
  const size_t s1 = pick_staged(false);
  const size_t s3 = pick_staged(true);

  // ---- carve
  Arena a(base);
  p.guards.clear();
  if (cfg.flags & LQSGD_FLAG_GUARD_WORDS) a.guards = &p.guards;
  p.d_layers = a.take<LayerDev>(p.mats.size());
  p.d_vecs = a.take<VectorDev>(p.vecs.size());
  p.state_begin = align_up(a.off, 256);
  p.layers.resize(p.mats.size());
  for (size_t li = 0; li < p.mats.size(); ++li) {
    const MatHost& mt = p.mats[li];
    LayerDev& L = p.layers[li];
    std::memset(&L, 0, sizeof(L));
    L.n = mt.n; L.m = mt.m; L.r = mt.r; L.vec = vec_of(mt.m) == 4; L.user_index = mt.user_index;
    const bool st = staged(mt), tc = on_tc(mt), pl = plain(mt);
    const auto scols = staged_cols(mt.m);
    const int cw = chunk_width(mt.m, c1);
    // pass 2: register path, or tensor cores (row chunks in multiples of the 64 rows of an operand slot)
    const int tr2 = tc ? (int)align_up((size_t)balanced_rows(mt.n, kTcRowChunk), 64) : balanced_rows(mt.n, r2);
    // tensor-core pass 1: column chunks balanced in units of 32 columns, at most kTcPass1Cols wide
    const int tc_units = ceil_div(mt.m, 32), tc_ncc = ceil_div(tc_units * 32, kTcPass1Cols);
    L.ncc = p.resident ? res_ncc[li] : (tc ? tc_ncc : (st ? (int)scols.size() : (pl ? 1 : ceil_div(mt.m, cw))));
    L.nrb = p.resident ? res_nrb[li] : ceil_div(mt.n, tr2);
    L.npb = ceil_div(mt.n, kFactorBlockRows);
    L.nqb = ceil_div(mt.m, kFactorBlockRows);
    L.qfused = (tc && L.nrb == 1 && !colscales && !p.resident) ? 1 : 0;
    const size_t nm = (size_t)mt.n * mt.m;
    L.E = a.take<float>((size_t)W * nm);
    L.Q = a.take<float>((size_t)mt.m * RP);
    L.mt = (int)align_up((size_t)mt.m, 4);
    L.tc = tc ? 1 : 0;
    if (tc) p.any_tc = true;
    L.nt = (int)align_up((size_t)mt.n, 4);
    L.Qt = a.take<float>((size_t)(tc ? 2 : 1) * RP * L.mt);
    L.Pbt = tc ? a.take<float>((size_t)3 * RP * L.nt) : nullptr;
    L.kcat = (int)align_up((size_t)3 * RP, 32);
    L.Pcat = tc ? a.take<float>((size_t)mt.n * L.kcat) : nullptr;
    L.Qcat = tc ? a.take<float>((size_t)mt.m * L.kcat) : nullptr;
    L.Ppart = a.take<float>((size_t)W * L.ncc * mt.n * RP);
    L.Praw = (L.ncc == 1) ? L.Ppart : a.take<float>((size_t)W * mt.n * RP);
    L.P = a.take<float>((size_t)W * mt.n * RP);
    L.Pbar = a.take<float>((size_t)mt.n * RP);
    L.Qpart = a.take<float>((size_t)W * L.nrb * mt.m * RP);
    L.Qw = (L.nrb == 1) ? L.Qpart : a.take<float>((size_t)W * mt.m * RP);
    L.gram_part = a.take<double>((size_t)W * L.npb * RP * RP);
    L.chol = RP >= kCholSplitRP ? a.take<double>((size_t)W * (RP * RP + 2 * RP)) : nullptr;
    // many partial sums: folded in groups first (fold_kernel), the steps then add the groups' sums
    auto fold = [&](std::vector<FoldJob>& jobs, const void* src, int nparts, size_t plane, bool dbl, int& nsum) -> const void* {
      nsum = nparts;
      if (p.resident || nparts <= kFoldAbove) return src;
      const int ng = ceil_div(nparts, kFoldGroup);
      const size_t esz = dbl ? sizeof(double) : sizeof(float);
      unsigned char* dst = dbl ? reinterpret_cast<unsigned char*>(a.take<double>((size_t)W * ng * plane))
                               : reinterpret_cast<unsigned char*>(a.take<float>((size_t)W * ng * plane));
      for (int w = 0; w < W; ++w)
        for (int g = 0; g < ng; ++g)
          for (size_t e0 = 0; e0 < plane; e0 += kFoldElems)
            jobs.push_back({static_cast<const unsigned char*>(src) + ((size_t)w * nparts + (size_t)g * kFoldGroup) * plane * esz,
                            dst + ((size_t)w * ng + g) * plane * esz, (uint32_t)plane, (uint32_t)e0,
                            (uint16_t)std::min(kFoldGroup, nparts - g * kFoldGroup), (uint16_t)(dbl ? 1 : 0), 0u});
      nsum = ng;
      return dst;
    };
    L.Psum = static_cast<const float*>(fold(p.foldP, L.Ppart, L.ncc, (size_t)mt.n * RP, false, L.nps));
    L.Qsum = static_cast<const float*>(fold(p.foldQ, L.Qpart, L.nrb, (size_t)mt.m * RP, false, L.nqs));
    L.gram_sum = static_cast<const double*>(fold(p.foldG, L.gram_part, L.npb, (size_t)RP * RP, true, L.ngs));
    L.maxp = a.take<float>((size_t)W * L.npb * (colscales ? RP : 1));
    L.maxq = a.take<float>((size_t)W * L.nqb * (colscales ? RP : 1));
    L.scales = a.take<float>(2 * (size_t)RP);
    const auto& lo = p.layout[mt.user_index];
    L.pay_scale_off = lo.scale_offset; L.pay_p_off = lo.p_offset; L.pay_q_off = lo.q_offset;

    // tiles
    const int li32 = (int)li;
    if (st) {
      const int tr1 = tile_rows(mt.n, mt.m, s1, 1), tr3 = tile_rows(mt.n, mt.m, std::max<size_t>(s3, 1), 1);
      for (int rb = 0; rb < ceil_div(mt.n, tr1); ++rb)
        for (int cc = 0; cc < (int)scols.size(); ++cc)
          for (int w = 0; w < W; ++w)
            p.stiles1.push_back({li32, w, rb * tr1, std::min(tr1, mt.n - rb * tr1), scols[cc].first, scols[cc].second, cc, 0});
      for (int rb = 0; rb < ceil_div(mt.n, tr3); ++rb)
        for (int cc = 0; cc < (int)scols.size(); ++cc)
          p.stiles3.push_back({li32, 0, rb * tr3, std::min(tr3, mt.n - rb * tr3), scols[cc].first, scols[cc].second, 0, 0});
    }
    if (pl) {
      for (int rb = 0; rb < ceil_div(mt.n, kStreamPlainRows); ++rb) {
        const int row0 = rb * kStreamPlainRows, nrows = std::min(kStreamPlainRows, mt.n - row0);
        for (int w = 0; w < W; ++w) p.stiles1.push_back({li32, w, row0, nrows, 0, mt.m, 0, 1});
        p.stiles3.push_back({li32, 0, row0, nrows, 0, mt.m, 0, 1});
      }
    }
    if (tc) {
      int u0 = 0;
      for (int cc = 0; cc < tc_ncc; ++cc) {
        const int nu = tc_units / tc_ncc + (cc < tc_units % tc_ncc ? 1 : 0);
        const int col0 = u0 * 32, ncols = std::min(nu * 32, mt.m - col0);
        for (int rb = 0; rb < ceil_div(mt.n, kTcRowsPerTile); ++rb)
          for (int w = 0; w < W; ++w)
            p.tctiles1.push_back({li32, w, rb * kTcRowsPerTile, std::min(kTcRowsPerTile, mt.n - rb * kTcRowsPerTile), col0, ncols, cc, 0});
        u0 += nu;
      }
    }
    for (int rb = 0; tc && rb < ceil_div(mt.n, kTcRowsPerTile); ++rb)
      for (int cb = 0; cb < ceil_div(mt.m, 128); ++cb)
        p.tctiles3.push_back({li32, 0, rb * kTcRowsPerTile, std::min(kTcRowsPerTile, mt.n - rb * kTcRowsPerTile), cb * 128,
                              std::min(128, mt.m - cb * 128), 0, 0});
    for (int rb = 0; !p.resident && !st && !tc && !pl && rb < ceil_div(mt.n, kPass1Rows); ++rb)
      for (int cc = 0; cc < L.ncc; ++cc)
        for (int w = 0; w < W; ++w) {
          const int row0 = rb * kPass1Rows, col0 = cc * cw;
          p.tiles1.push_back({li32, w, row0, std::min(kPass1Rows, mt.n - row0), col0, std::min(cw, mt.m - col0), cc, 0});
        }
    const int cw2 = 128 * vec_of(mt.m);
    for (int w = 0; w < W; ++w)
      for (int rb = 0; rb < L.nrb; ++rb)
        for (int cc = 0; cc < ceil_div(mt.m, cw2); ++cc) {
          const int row0 = rb * tr2, col0 = cc * cw2;
          if (tc || p.resident) continue;
          p.tiles2.push_back({li32, w, row0, std::min(tr2, mt.n - row0), col0, std::min(cw2, mt.m - col0), rb, 0});
        }
    for (int w = 0; tc && w < W; ++w)
      for (int rb = 0; rb < L.nrb; ++rb)
        for (int cc = 0; cc < ceil_div(mt.m, 128); ++cc) {
          const int row0 = rb * tr2, col0 = cc * 128;
          p.tctiles2.push_back({li32, w, row0, std::min(tr2, mt.n - row0), col0, std::min(128, mt.m - col0), rb, 0});
        }
    const int tr3 = balanced_rows(mt.n, r3);
    for (int rb = 0; !p.resident && !st && !tc && !pl && rb < ceil_div(mt.n, tr3); ++rb)
      for (int cc = 0; cc < ceil_div(mt.m, cw2); ++cc) {
        const int row0 = rb * tr3, col0 = cc * cw2;
        p.tiles3.push_back({li32, 0, row0, std::min(tr3, mt.n - row0), col0, std::min(cw2, mt.m - col0), 0, 0});
      }
    const bool one_cta = RP <= 8 && mt.n <= kOrthSmallMaxRows;
    for (int w = 0; w < W; ++w) {
      if (one_cta) p.fbS.push_back({li32, w, 0, 0});
      if (!one_cta && RP >= kCholSplitRP) p.fbC.push_back({li32, w, 0, 0});
      for (int b = 0; !one_cta && b < L.npb; ++b) p.fbP.push_back({li32, w, b, 0});
      for (int b = 0; !L.qfused && b < L.nqb; ++b) p.fbQ.push_back({li32, w, b, 0});
    }
    for (int c = 0; c < ceil_div(mt.n * mt.r, kExchangeChunk); ++c) p.chP.push_back({li32, c});
    for (int c = 0; c < ceil_div(mt.m * mt.r, kExchangeChunk); ++c) p.chQ.push_back({li32, c});
  }
  for (size_t vi = 0; vi < p.vecs.size(); ++vi)
    for (int c = 0; c < ceil_div(p.vecs[vi].len, 256); ++c) p.chV.push_back({(int)vi, c});
  // Pass 2 walks the data in the reverse of pass 1's order and pass 3 again in pass 1's order:
  // each pass starts on what the previous one touched last, which is still in L2.
  std::reverse(p.tiles2.begin(), p.tiles2.end());
  // Tensor-core pass 2 deals its tiles round-robin to one CTA per SM: tallest first, so the CTAs finish together.
  std::stable_sort(p.tctiles2.begin(), p.tctiles2.end(), [](const Tile& x, const Tile& y) { return x.nrows > y.nrows; });
  // Pass 1 hands its tiles out at run time: widest first (a tile costs its column count: every stage is 128 rows
  // deep whatever the tile's row count), so that the short ones fill the end.
  p.tc_grid = sm_count;
  std::stable_sort(p.tctiles1.begin(), p.tctiles1.end(), [](const Tile& x, const Tile& y) { return x.ncols > y.ncols; });
  // Pass 3 hands its tiles out at run time, in table order (CTAs that walk neighbouring tiles at the same time are
  // what the memory likes: contiguous shares of the list per CTA ran 11 % slower).  A tile with all its workers is
  // a megabyte and more, too coarse a unit for an even finish: its workers are cut into ranges [worker, part) so
  // that there are about a dozen units per SM; every unit forms the tile's G_hat itself (the factors are small),
  // the one that has worker 0 writes it.
  {
    const std::vector<Tile> in = p.tctiles3;
    const size_t want_units = (size_t)12 * p.tc_grid;
    const int per = (int)std::max<size_t>(1, std::min<size_t>((size_t)W, in.size() * (size_t)W / std::max<size_t>(1, want_units)));
    const int nr = ceil_div(W, per);             // ranges per tile, of nearly equal size
    p.tctiles3.clear();
    for (const Tile& tl : in)
      for (int r = 0; r < nr; ++r) {
        Tile e = tl;
        e.worker = (int)((long)W * r / nr);
        e.part = (int)((long)W * (r + 1) / nr);
        p.tctiles3.push_back(e);
      }
  }
  p.d_status = a.take<uint32_t>(p.mats.size());
  p.d_stats = a.take<unsigned long long>(4);
  p.d_payload = a.take<uint8_t>((size_t)W * p.payload_stride);
  p.xscale_ns = colscales ? RP : 1;
  p.d_xscales = a.take<float>(2 * p.mats.size() * p.xscale_ns);
  p.vec_elems = 0;
  for (auto& v : p.vecs) p.vec_elems += (size_t)v.len;
  p.vec_pay_base = p.vecs.empty() ? 0 : p.vecs.front().pay_off;
  p.d_xvec = a.take<float>(p.vec_elems);
  p.d_xsend[0] = a.take<uint8_t>((size_t)W * p.region_bytes[0]);
  p.d_xsend[1] = a.take<uint8_t>((size_t)W * p.region_bytes[1]);
  p.d_rsync = a.take<uint32_t>(1 + 2 * kResBarriers);
  p.d_tcsched = a.take<int>(2 * 3);              // per tensor-core pass: draw counter, CTAs that have left (zero between launches)
  p.d_rstamps = a.take<uint64_t>(kResStamps + 1);
  p.state_end = a.off;

  // value-domain average: the table of one worker's dequantised levels serves every worker
  const int table_w = (cfg.flags & LQSGD_FLAG_AVERAGE_VALUES) ? 1 : p.W_total;
  quant_tables(cfg.bits_p, cfg.alpha, table_w, p.thrP, p.deqP);
  quant_tables(cfg.bits_q, cfg.alpha, table_w, p.thrQ, p.deqQ);
  p.d_tiles1 = a.take<Tile>(p.tiles1.size());
  p.d_tiles2 = a.take<Tile>(p.tiles2.size());
  p.d_tiles3 = a.take<Tile>(p.tiles3.size());
  p.d_stiles1 = a.take<Tile>(p.stiles1.size());
  p.d_stiles3 = a.take<Tile>(p.stiles3.size());
  p.d_tctiles2 = a.take<Tile>(p.tctiles2.size());
  p.d_tctiles1 = a.take<Tile>(p.tctiles1.size());
  p.d_tctiles3 = a.take<Tile>(p.tctiles3.size());
  p.d_tcmaps = a.take<uint8_t>(p.mats.size() * kTcMapsPerLayer * kTcMapBytes);
  p.d_rtiles = a.take<ResTile>(p.rtiles.size());
  p.d_rbegin = a.take<int>(p.rbegin.size());
  p.d_fbP = a.take<FactorBlock>(p.fbP.size());
  p.d_fbQ = a.take<FactorBlock>(p.fbQ.size());
  p.d_fbS = a.take<FactorBlock>(p.fbS.size());
  p.d_fbC = a.take<FactorBlock>(p.fbC.size());
  p.d_foldP = a.take<FoldJob>(p.foldP.size());
  p.d_foldG = a.take<FoldJob>(p.foldG.size());
  p.d_foldQ = a.take<FoldJob>(p.foldQ.size());
  p.d_chP = a.take<ExchangeChunk>(p.chP.size());
  p.d_chQ = a.take<ExchangeChunk>(p.chQ.size());
  p.d_chV = a.take<ExchangeChunk>(p.chV.size());
  p.d_thrP = a.take<float>(p.thrP.size());
  p.d_thrQ = a.take<float>(p.thrQ.size());
  p.d_deqP = a.take<float>(p.deqP.size());
  p.d_deqQ = a.take<float>(p.deqQ.size());
  p.d_ptrs = a.take<void*>(kPtrSets * (p.mats.size() + p.vecs.size()) * (size_t)(W + 2));
  if (p.any_tc) p.d_gmaps = a.take<uint8_t>(kPtrSets * p.mats.size() * (size_t)W * kTcMapBytes);
  if (cfg.power_iters > 1) {
    size_t big = 0;
    for (auto& mt : p.mats) big = std::max(big, (size_t)mt.n * mt.m);
    p.zero_elems = big;
    p.d_zero_ptrs = a.take<void*>(p.mats.size() * (size_t)W);
    if (p.any_tc) p.d_zero_gmaps = a.take<uint8_t>(p.mats.size() * (size_t)W * kTcMapBytes);
    p.d_zero = a.take<float>(big);
  }
  if (cfg.flags & LQSGD_FLAG_HOST_STAGING) {
    p.d_stage_g = a.take<float>((size_t)W * p.elems_total);
    p.d_stage_ghat = a.take<float>(p.elems_total);
  }
  if (a.guards) {                                   // the table of guard offsets itself, and the check's result
    a.guards = nullptr;
    p.d_guards = a.take<uint64_t>(p.guards.size());
    p.d_guard_result = a.take<unsigned long long>(2);
  }
  p.bytes = align_up(a.off, 256);
}

// Q_0 ~ N(0,1) (Alg. 1 initialisation): counter-based, a 64-bit integer mix of
// (seed, layer, element) feeding Box-Muller in double precision.
uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}
float normal_draw(uint64_t seed, uint64_t layer, uint64_t idx) {
  const uint64_t k = mix64(mix64(seed ^ 0xA0761D6478BD642Full) + layer * 0xE7037ED1A0B428DBull);
  const uint64_t a = mix64(k + 2 * idx), b = mix64(k + 2 * idx + 1);
  const double u1 = ((double)(a >> 11) + 1.0) * (1.0 / 9007199254740992.0);   // (0, 1]
  const double u2 = (double)(b >> 11) * (1.0 / 9007199254740992.0);           // [0, 1)
  return (float)(std::sqrt(-2.0 * std::log(u1)) * std::cos(6.283185307179586476925 * u2));
}

}  // namespace

struct lqsgd_ctx {
  lqsgd_config cfg;
  std::vector<lqsgd_shape> shapes;
  Plan plan;
  int device = 0, sm_count = 0;
  int grid1 = 0, grid2 = 0, grid3 = 0;
  std::vector<std::vector<void*>> ptr_sets;   // host mirrors of the device pointer tables (empty: slot unused)
  std::vector<uint64_t> ptr_used;             // last use of each slot (step counter), for eviction
  std::vector<char> ptr_pinned;               // slot was used by a capturing stream: a graph may replay it, never evicted
  uint64_t step_counter = 0;
  size_t ptr_count = 0;                       // pointers per table
  void** ptrs_cur = nullptr;                  // the device table of the current step
  void* workspace = nullptr;
  cudaEvent_t phase_events[LQSGD_N_PHASES + 1];
  bool have_events = false;
  Tables tables{};                   // filled by prepare_step
  bool has_weights = false;
  int round_stage = 0;               // progress of a split round (lqsgd_round_*)
  uint32_t test_wait_limit = 0;      // lqsgd_test_expire_wait: applies to the next step, then cleared
  int test_skip_pass = 0, test_skip_stage = 0;
  // A layer set whose passes run as a big kernel (staged or tensor-core) plus a register kernel for a few small layers
  // with unaligned rows: the register kernel goes to a stream of its own, forked from and joined to the caller's
  // around every pass, so that it runs beside the big kernel instead of in front of it (5 to 17 us per pass).
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  ~lqsgd_ctx() {
    if (ev_fork) cudaEventDestroy(ev_fork);
    if (ev_join) cudaEventDestroy(ev_join);
    if (side) cudaStreamDestroy(side);
  }
};

// The fp32 1-D tensors need no kernel of their own when the fused exchange of P runs anyway: their blocks (same
// shape) are appended to that launch.  Not in a split round (its exchange only packs), not in the quantised variant.
static bool vectors_ride(const lqsgd_ctx* c) {
  const bool quantised = (c->cfg.flags & LQSGD_FLAG_QUANTIZE_VECTORS) && c->cfg.bits_p != 32;
  return !c->plan.mats.empty() && !c->plan.chV.empty() && !quantised && c->plan.W_total == c->plan.W;
}

extern "C" {

int lqsgd_version(void) { return LQSGD_VERSION; }

const char* lqsgd_last_cuda_error(void) { return g_cuda_error.c_str(); }

const char* lqsgd_strerror(int code) {
  switch (code) {
    case LQSGD_OK: return "ok";
    case LQSGD_ERR_INVALID_ARG: return "invalid argument";
    case LQSGD_ERR_BAD_SHAPE: return "bad layer shape";
    case LQSGD_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case LQSGD_ERR_MISALIGNED: return "misaligned pointer";
    case LQSGD_ERR_CUDA: return "CUDA runtime error";
    case LQSGD_ERR_NO_STAGING: return "context was created without host staging";
    case LQSGD_ERR_OUT_OF_RANGE: return "index out of range";
    case LQSGD_ERR_TOO_LARGE: return "size exceeds the built-in scratch of the no-allocation entry point";
    case LQSGD_ERR_CAPTURE: return "stream is capturing and the tensor pointers changed since the previous call";
    case LQSGD_ERR_PLAN: return "the work tables of this configuration fail an invariant (lqsgd_plan_check)";
    default: return "unknown error";
  }
}

int lqsgd_workspace_bytes(const lqsgd_shape* shapes, int32_t n_layers, const lqsgd_config* cfg, size_t* out) {
  if (!out) return LQSGD_ERR_INVALID_ARG;
  const int rc = check_config(shapes, n_layers, cfg);
  if (rc != LQSGD_OK) return rc;
  Plan p;
  // The size must not depend on the device: plan for the largest SM count tile sizes consider.
  make_plan(shapes, n_layers, *cfg, nullptr, 148, p);
  Plan p2, p3;
  make_plan(shapes, n_layers, *cfg, nullptr, 1, p2);
  make_plan(shapes, n_layers, *cfg, nullptr, 148, p3, false);     // in case the one-launch round cannot run on the device
  *out = std::max({p.bytes, p2.bytes, p3.bytes});
  return LQSGD_OK;
}

namespace {
// lqsgd_plan_check: the invariants of a plan.  Every tiling here is a grid (row bands cut into column chunks), so
// "covers once" is checked band by band.
struct Rect { int row0, nrows, col0, ncols, part; };
std::string check_grid(std::vector<Rect> v, int n, int m, int nparts, bool parts_along_cols, const char* what) {
  // rows: bands in order, contiguous from 0 to n; inside a band the chunks contiguous from 0 to m
  std::sort(v.begin(), v.end(), [](const Rect& a, const Rect& b) { return a.row0 != b.row0 ? a.row0 < b.row0 : a.col0 < b.col0; });
  std::map<int, std::vector<int>> parts_of;       // chunk position along the OTHER axis -> parts seen
  size_t i = 0;
  int row = 0;
  while (i < v.size()) {
    if (v[i].row0 != row) return std::string(what) + ": row band does not start where the last ended";
    const int nr = v[i].nrows;
    if (nr < 1) return std::string(what) + ": empty tile";
    int col = 0;
    for (; i < v.size() && v[i].row0 == row; ++i) {
      if (v[i].nrows != nr) return std::string(what) + ": tiles of one band differ in height";
      if (v[i].col0 != col || v[i].ncols < 1) return std::string(what) + ": column chunk does not start where the last ended";
      col += v[i].ncols;
      if (nparts > 0) {
        if (v[i].part < 0 || v[i].part >= nparts) return std::string(what) + ": partial-sum index out of range";
        parts_of[parts_along_cols ? row : v[i].col0].push_back(v[i].part);
      }
    }
    if (col != m) return std::string(what) + ": a band's chunks do not end at the last column";
    row += nr;
  }
  if (row != n) return std::string(what) + ": bands do not end at the last row";
  for (auto& kv : parts_of) {                      // every partial sum written exactly once
    std::vector<int>& ps = kv.second;
    std::sort(ps.begin(), ps.end());
    if ((int)ps.size() != nparts) return std::string(what) + ": partial sums written != partial sums added up";
    for (int k = 0; k < nparts; ++k)
      if (ps[k] != k) return std::string(what) + ": a partial sum is written twice or never";
  }
  return "";
}

std::string check_plan(const Plan& p) {
  const int W = p.W;
  const size_t nm = p.mats.size();
  auto layer_name = [&](size_t li) { return " (layer " + std::to_string(p.mats[li].user_index) + ", " + std::to_string(p.mats[li].n) + " x " + std::to_string(p.mats[li].m) + ")"; };
  // ---- passes 1 and 2: per (layer, worker) one grid; pass 3: per layer one grid over all workers
  std::vector<std::vector<Rect>> g1(nm * W), g2(nm * W), g3(nm);
  std::map<std::array<int, 3>, std::vector<std::pair<int, int>>> tc3;     // (layer, row0, col0) -> worker ranges
  auto bad_tile = [&](const Tile& tl) { return tl.layer < 0 || tl.layer >= (int)nm || tl.worker < 0 || tl.worker >= W; };
  for (auto* list : {&p.tiles1, &p.stiles1, &p.tctiles1})
    for (const Tile& tl : *list) {
      if (bad_tile(tl)) return "pass 1: tile with a layer or worker out of range";
      g1[(size_t)tl.layer * W + tl.worker].push_back({tl.row0, tl.nrows, tl.col0, tl.ncols, tl.part});
    }
  for (auto* list : {&p.tiles2, &p.tctiles2})
    for (const Tile& tl : *list) {
      if (bad_tile(tl)) return "pass 2: tile with a layer or worker out of range";
      g2[(size_t)tl.layer * W + tl.worker].push_back({tl.row0, tl.nrows, tl.col0, tl.ncols, tl.part});
    }
  for (auto* list : {&p.tiles3, &p.stiles3})
    for (const Tile& tl : *list) {
      if (tl.layer < 0 || tl.layer >= (int)nm) return "pass 3: tile with a layer out of range";
      g3[tl.layer].push_back({tl.row0, tl.nrows, tl.col0, tl.ncols, 0});
    }
  for (const Tile& tl : p.tctiles3) {
    if (tl.layer < 0 || tl.layer >= (int)nm) return "pass 3: tile with a layer out of range";
    auto& ranges = tc3[{tl.layer, tl.row0, tl.col0}];
    if (ranges.empty()) g3[tl.layer].push_back({tl.row0, tl.nrows, tl.col0, tl.ncols, 0});
    ranges.push_back({tl.worker, tl.part});
  }
  for (auto& kv : tc3) {                           // a tile's ranges of workers: 0 .. W without gap or overlap
    auto r = kv.second;
    std::sort(r.begin(), r.end());
    int w = 0;
    for (auto& ab : r) {
      if (ab.first != w || ab.second <= ab.first) return "pass 3: a tile's ranges of workers leave a gap or overlap" + layer_name(kv.first[0]);
      w = ab.second;
    }
    if (w != W) return "pass 3: a tile's ranges of workers do not end at the last worker" + layer_name(kv.first[0]);
  }
  if (p.resident) {
    for (const ResTile& tl : p.rtiles) {
      if (tl.layer < 0 || tl.layer >= (int)nm || tl.worker < 0 || tl.worker >= W) return "one-launch round: tile out of range";
      g1[(size_t)tl.layer * W + tl.worker].push_back({tl.row0, tl.nrows, tl.col0, tl.ncols, tl.part_c});
      g2[(size_t)tl.layer * W + tl.worker].push_back({tl.row0, tl.nrows, tl.col0, tl.ncols, tl.part_r});
      if (tl.worker == 0) g3[tl.layer].push_back({tl.row0, tl.nrows, tl.col0, tl.ncols, 0});
      if ((tl.worker == 0) != (tl.writes_ghat != 0)) return "one-launch round: G_hat is written by worker 0's tiles, and only those";
    }
  }
  for (size_t li = 0; li < nm; ++li) {
    const LayerDev& L = p.layers[li];
    for (int w = 0; w < W; ++w) {
      std::string e = check_grid(g1[li * W + w], L.n, L.m, L.ncc, true, "pass 1");
      if (e.empty()) e = check_grid(g2[li * W + w], L.n, L.m, L.nrb, false, "pass 2");
      if (!e.empty()) return e + layer_name(li) + ", worker " + std::to_string(w);
    }
    std::string e = check_grid(g3[li], L.n, L.m, 0, true, "pass 3");
    if (!e.empty()) return e + layer_name(li);
    if (L.npb != ceil_div(L.n, kFactorBlockRows) || L.nqb != ceil_div(L.m, kFactorBlockRows)) return "factor block counts" + layer_name(li);
  }
  // ---- factor blocks and exchange chunks
  {
    std::vector<int> seenP(nm * W, 0), seenQ(nm * W, 0), seenS(nm * W, 0);
    std::map<std::pair<size_t, int>, int> blkP, blkQ;
    for (const FactorBlock& f : p.fbS) { if (f.layer < 0 || f.layer >= (int)nm || f.worker < 0 || f.worker >= W) return "Orthonormalize: block out of range"; ++seenS[(size_t)f.layer * W + f.worker]; }
    for (const FactorBlock& f : p.fbP) { if (f.layer < 0 || f.layer >= (int)nm || f.worker < 0 || f.worker >= W) return "Orthonormalize: block out of range"; ++blkP[{(size_t)f.layer * W + f.worker, f.blk}]; }
    for (const FactorBlock& f : p.fbQ) { if (f.layer < 0 || f.layer >= (int)nm || f.worker < 0 || f.worker >= W) return "Q_w reduction: block out of range"; ++blkQ[{(size_t)f.layer * W + f.worker, f.blk}]; }
    for (size_t li = 0; li < nm; ++li)
      for (int w = 0; w < W; ++w) {
        const size_t k = li * W + w;
        const LayerDev& L = p.layers[li];
        int np = 0;
        for (int b = 0; b < L.npb; ++b) { auto it = blkP.find({k, b}); if (it != blkP.end()) { if (it->second != 1) return "Orthonormalize: a block of rows twice" + layer_name(li); ++np; } }
        if (!((seenS[k] == 1 && np == 0) || (seenS[k] == 0 && np == L.npb))) return "Orthonormalize: every row of P once, by one CTA or by blocks of 128" + layer_name(li);
        for (int b = 0; b < L.nqb; ++b) {
          auto it = blkQ.find({k, b});
          if (L.qfused ? it != blkQ.end() : (it == blkQ.end() || it->second != 1)) return "Q_w reduction: every block of 128 rows of Q once, or none where pass 2 takes the maxima" + layer_name(li);
        }
        if (L.qfused && (!L.tc || L.nrb != 1)) return "Q_w maxima in pass 2 need the whole sum in one tile" + layer_name(li);
      }
    if (blkP.size() + 0 != [&] { size_t t = 0; for (size_t li = 0; li < nm; ++li) for (int w = 0; w < W; ++w) if (!seenS[li * W + w]) t += p.layers[li].npb; return t; }()) return "Orthonormalize: blocks beyond the layers' rows";
    std::vector<std::vector<int>> cP(nm), cQ(nm);
    for (const ExchangeChunk& c : p.chP) { if (c.layer < 0 || c.layer >= (int)nm) return "exchange of P: chunk out of range"; cP[c.layer].push_back(c.chunk); }
    for (const ExchangeChunk& c : p.chQ) { if (c.layer < 0 || c.layer >= (int)nm) return "exchange of Q: chunk out of range"; cQ[c.layer].push_back(c.chunk); }
    for (size_t li = 0; li < nm; ++li) {
      const LayerDev& L = p.layers[li];
      auto full = [&](std::vector<int>& c, int elems) {
        std::sort(c.begin(), c.end());
        if ((int)c.size() != ceil_div(elems, kExchangeChunk)) return false;
        for (int k = 0; k < (int)c.size(); ++k) if (c[k] != k) return false;
        return true;
      };
      if (!full(cP[li], L.n * L.r) || !full(cQ[li], L.m * L.r)) return "exchange: every 256 factor elements once" + layer_name(li);
    }
  }
  // ---- second-level sums: every partial of a folded layer in exactly one group, every element of the plane once
  auto check_fold = [&](const std::vector<FoldJob>& jobs, const char* what, auto src_of, auto dst_of, auto nparts_of, auto nsum_of,
                        auto plane_of, size_t esz) -> std::string {
    std::map<std::tuple<size_t, int, int>, std::vector<std::pair<uint32_t, int>>> seen;   // (layer, worker, group) -> (e0, count)
    for (const FoldJob& j : jobs) {
      bool placed = false;
      for (size_t li = 0; li < nm && !placed; ++li) {
        const int nparts = nparts_of(li), ng = nsum_of(li);
        if (ng == nparts) continue;                                      // not folded
        const size_t plane = plane_of(li);
        const unsigned char* s0 = static_cast<const unsigned char*>(src_of(li));
        const unsigned char* d0 = static_cast<const unsigned char*>(dst_of(li));
        const unsigned char* js = static_cast<const unsigned char*>(j.src);
        if (js < s0 || js >= s0 + (size_t)W * nparts * plane * esz) continue;
        const size_t part_index = (size_t)(js - s0) / (plane * esz);
        if ((size_t)(js - s0) % (plane * esz)) return std::string(what) + ": a group does not start on a partial sum";
        const int w = (int)(part_index / nparts), first = (int)(part_index % nparts);
        if (first % kFoldGroup) return std::string(what) + ": a group does not start on a multiple of the group size";
        const int g = first / kFoldGroup;
        if (j.count != std::min(kFoldGroup, nparts - first) || j.plane != plane || (j.is_double != 0) != (esz == 8))
          return std::string(what) + ": a group's extent is wrong";
        if (static_cast<unsigned char*>(j.dst) != d0 + ((size_t)w * ng + g) * plane * esz) return std::string(what) + ": a group's sum goes to the wrong place";
        seen[{li, w, g}].push_back({j.e0, 0});
        placed = true;
      }
      if (!placed) return std::string(what) + ": a job outside every folded layer";
    }
    for (size_t li = 0; li < nm; ++li) {
      const int nparts = nparts_of(li), ng = nsum_of(li);
      if (ng == nparts) { if (nparts > kFoldAbove && !p.resident) return std::string(what) + ": a layer with many partial sums is not folded"; continue; }
      if (ng != ceil_div(nparts, kFoldGroup)) return std::string(what) + ": group count";
      for (int w = 0; w < W; ++w)
        for (int g = 0; g < ng; ++g) {
          auto it = seen.find({li, w, g});
          if (it == seen.end()) return std::string(what) + ": a group is never summed" + layer_name(li);
          auto& v = it->second;
          std::sort(v.begin(), v.end());
          uint32_t e = 0;
          for (auto& x : v) { if (x.first != e) return std::string(what) + ": a plane's elements twice or never" + layer_name(li); e += kFoldElems; }
          if (e < plane_of(li)) return std::string(what) + ": a plane's last elements are never summed" + layer_name(li);
        }
    }
    return "";
  };
  {
    std::string e = check_fold(p.foldP, "fold of P partials", [&](size_t li) { return (const void*)p.layers[li].Ppart; },
                               [&](size_t li) { return (const void*)p.layers[li].Psum; }, [&](size_t li) { return p.layers[li].ncc; },
                               [&](size_t li) { return p.layers[li].nps; }, [&](size_t li) { return (size_t)p.layers[li].n * p.RP; }, 4);
    if (e.empty())
      e = check_fold(p.foldQ, "fold of Q partials", [&](size_t li) { return (const void*)p.layers[li].Qpart; },
                     [&](size_t li) { return (const void*)p.layers[li].Qsum; }, [&](size_t li) { return p.layers[li].nrb; },
                     [&](size_t li) { return p.layers[li].nqs; }, [&](size_t li) { return (size_t)p.layers[li].m * p.RP; }, 4);
    if (e.empty())
      e = check_fold(p.foldG, "fold of block Grams", [&](size_t li) { return (const void*)p.layers[li].gram_part; },
                     [&](size_t li) { return (const void*)p.layers[li].gram_sum; }, [&](size_t li) { return p.layers[li].npb; },
                     [&](size_t li) { return p.layers[li].ngs; }, [&](size_t li) { return (size_t)p.RP * p.RP; }, 8);
    if (!e.empty()) return e;
  }
  return "";
}
}  // namespace

static thread_local int g_plan_defect = 0;
int lqsgd_test_plan_defect(int32_t kind) {
  if (kind < 0 || kind > 5) return LQSGD_ERR_INVALID_ARG;
  g_plan_defect = kind;
  return LQSGD_OK;
}

int lqsgd_plan_check(const lqsgd_shape* shapes, int32_t n_layers, const lqsgd_config* cfg, int32_t sm_count, char* msg,
                     size_t msg_len) {
  if (msg && msg_len) msg[0] = 0;
  const int rc = check_config(shapes, n_layers, cfg);
  if (rc != LQSGD_OK) return rc;
  if (sm_count < 1 || sm_count > 1024) return LQSGD_ERR_INVALID_ARG;
  // a base address that keeps every piece's address distinct and non-null (nothing is dereferenced)
  std::vector<std::string> found;
  for (int allow_resident = 1; allow_resident >= 0; --allow_resident) {
    Plan p;
    make_plan(shapes, n_layers, *cfg, reinterpret_cast<void*>((uintptr_t)1 << 40), sm_count, p, allow_resident != 0);
    if (g_plan_defect) {                       // test support: see lqsgd_test_plan_defect
      const int kind = g_plan_defect;
      auto drop_last = [](auto& v) { if (!v.empty()) v.pop_back(); };
      if (kind == 1) { if (!p.tctiles1.empty()) drop_last(p.tctiles1); else if (!p.stiles1.empty()) drop_last(p.stiles1); else if (!p.tiles1.empty()) drop_last(p.tiles1); else drop_last(p.rtiles); }
      if (kind == 2) {
        auto& v = !p.tctiles2.empty() ? p.tctiles2 : p.tiles2;
        if (v.size() >= 2) {                   // two tiles of one (layer, worker, column chunk), if there are such
          for (size_t i = 1; i < v.size(); ++i)
            if (v[i].layer == v[0].layer && v[i].worker == v[0].worker && v[i].col0 == v[0].col0) { v[i].part = v[0].part; break; }
          if (p.layers[v[0].layer].nrb == 1) v[0].part = 1;
        }
      }
      if (kind == 3) { if (!p.tctiles3.empty()) drop_last(p.tctiles3); else if (!p.stiles3.empty()) drop_last(p.stiles3); else drop_last(p.tiles3); }
      if (kind == 4) { if (!p.foldQ.empty()) drop_last(p.foldQ); else if (!p.foldG.empty()) drop_last(p.foldG); else drop_last(p.foldP); }
      if (kind == 5) drop_last(p.chQ);
    }
    const std::string e = check_plan(p);
    if (!e.empty()) {
      if (msg && msg_len) { std::strncpy(msg, e.c_str(), msg_len - 1); msg[msg_len - 1] = 0; }
      g_plan_defect = 0;
      return LQSGD_ERR_PLAN;
    }
    if (!p.resident) break;                     // the same plan again
  }
  g_plan_defect = 0;
  return LQSGD_OK;
}

int lqsgd_create(const lqsgd_shape* shapes, int32_t n_layers, const lqsgd_config* cfg, void* dev_workspace,
                 size_t workspace_bytes, lqsgd_ctx** ctx_out) {
  if (!ctx_out) return LQSGD_ERR_INVALID_ARG;
  *ctx_out = nullptr;
  int rc = check_config(shapes, n_layers, cfg);
  if (rc != LQSGD_OK) return rc;
  if (!dev_workspace) return LQSGD_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(dev_workspace) % 256) return LQSGD_ERR_MISALIGNED;
  size_t need = 0;
  rc = lqsgd_workspace_bytes(shapes, n_layers, cfg, &need);
  if (rc != LQSGD_OK) return rc;
  if (workspace_bytes < need) return LQSGD_ERR_WORKSPACE_TOO_SMALL;

  lqsgd_ctx* c = new (std::nothrow) lqsgd_ctx();
  if (!c) return LQSGD_ERR_INVALID_ARG;
  struct Guard { lqsgd_ctx* c; ~Guard() { delete c; } } guard{c};
  c->cfg = *cfg;
  c->shapes.assign(shapes, shapes + n_layers);
  c->workspace = dev_workspace;
  CK(cudaGetDevice(&c->device));
  CK(cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device));
  // tile sizes for 148 or for 1 SM bound the workspace; use the device's count if it fits
  int sm_plan = c->sm_count;
  make_plan(shapes, n_layers, *cfg, dev_workspace, sm_plan, c->plan);
  if (c->plan.bytes > workspace_bytes) {
    c->plan = Plan();
    sm_plan = 148;
    make_plan(shapes, n_layers, *cfg, dev_workspace, sm_plan, c->plan);
  }
  if (c->plan.resident) {
    // the one-launch round needs its CTA (shared memory, registers) to fit an SM; else the multi-kernel round
    int grid = 0;
    const cudaError_t e = resident_max_grid(c->plan.RP, c->plan.res_smem, c->sm_count, &grid);
    if (e != cudaSuccess || grid == 0) {
      (void)cudaGetLastError();
      c->plan = Plan();
      make_plan(shapes, n_layers, *cfg, dev_workspace, sm_plan, c->plan, false);
    }
  }
  Plan& p = c->plan;
  if (p.bytes > workspace_bytes) return LQSGD_ERR_WORKSPACE_TOO_SMALL;
  if (!p.tiles1.empty() && (!p.stiles1.empty() || !p.tctiles1.empty())) {
    CK(cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking));
    CK(cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming));
  }

  char* base = static_cast<char*>(dev_workspace);
  CK(cudaMemset(base + p.state_begin, 0, p.state_end - p.state_begin));   // E_0 = 0, padding columns 0
  auto up = [&](void* dst, const void* src, size_t bytes) -> cudaError_t {
    return bytes ? cudaMemcpy(dst, src, bytes, cudaMemcpyHostToDevice) : cudaSuccess;
  };
  CK(up(p.d_layers, p.layers.data(), p.layers.size() * sizeof(LayerDev)));
  CK(up(p.d_vecs, p.vecs.data(), p.vecs.size() * sizeof(VectorDev)));
  CK(up(p.d_tiles1, p.tiles1.data(), p.tiles1.size() * sizeof(Tile)));
  CK(up(p.d_tiles2, p.tiles2.data(), p.tiles2.size() * sizeof(Tile)));
  CK(up(p.d_tiles3, p.tiles3.data(), p.tiles3.size() * sizeof(Tile)));
  CK(up(p.d_stiles1, p.stiles1.data(), p.stiles1.size() * sizeof(Tile)));
  CK(up(p.d_stiles3, p.stiles3.data(), p.stiles3.size() * sizeof(Tile)));
  CK(up(p.d_tctiles2, p.tctiles2.data(), p.tctiles2.size() * sizeof(Tile)));
  CK(up(p.d_tctiles1, p.tctiles1.data(), p.tctiles1.size() * sizeof(Tile)));
  CK(up(p.d_tctiles3, p.tctiles3.data(), p.tctiles3.size() * sizeof(Tile)));
  p.tcmaps.resize(p.mats.size() * kTcMapsPerLayer * kTcMapBytes + 1);
  rc = tc_encode_maps(p.layers.data(), (int)p.layers.size(), p.W, p.RP, p.tcmaps.data());
  if (rc != LQSGD_OK) { g_cuda_error = "cuTensorMapEncodeTiled failed or is not available"; return rc; }
  CK(up(p.d_tcmaps, p.tcmaps.data(), p.mats.size() * kTcMapsPerLayer * kTcMapBytes));
  if (!p.guards.empty()) {
    CK(up(p.d_guards, p.guards.data(), p.guards.size() * sizeof(uint64_t)));
    CK(launch_guards(base, p.d_guards, (int)p.guards.size(), kGuardPattern, nullptr, nullptr));
  }
  CK(up(p.d_rtiles, p.rtiles.data(), p.rtiles.size() * sizeof(ResTile)));
  CK(up(p.d_rbegin, p.rbegin.data(), p.rbegin.size() * sizeof(int)));
  CK(up(p.d_fbP, p.fbP.data(), p.fbP.size() * sizeof(FactorBlock)));
  CK(up(p.d_fbQ, p.fbQ.data(), p.fbQ.size() * sizeof(FactorBlock)));
  CK(up(p.d_fbS, p.fbS.data(), p.fbS.size() * sizeof(FactorBlock)));
  CK(up(p.d_fbC, p.fbC.data(), p.fbC.size() * sizeof(FactorBlock)));
  CK(up(p.d_foldP, p.foldP.data(), p.foldP.size() * sizeof(FoldJob)));
  CK(up(p.d_foldG, p.foldG.data(), p.foldG.size() * sizeof(FoldJob)));
  CK(up(p.d_foldQ, p.foldQ.data(), p.foldQ.size() * sizeof(FoldJob)));
  CK(up(p.d_chP, p.chP.data(), p.chP.size() * sizeof(ExchangeChunk)));
  CK(up(p.d_chQ, p.chQ.data(), p.chQ.size() * sizeof(ExchangeChunk)));
  CK(up(p.d_chV, p.chV.data(), p.chV.size() * sizeof(ExchangeChunk)));
  CK(up(p.d_thrP, p.thrP.data(), p.thrP.size() * sizeof(float)));
  CK(up(p.d_thrQ, p.thrQ.data(), p.thrQ.size() * sizeof(float)));
  CK(up(p.d_deqP, p.deqP.data(), p.deqP.size() * sizeof(float)));
  CK(up(p.d_deqQ, p.deqQ.data(), p.deqQ.size() * sizeof(float)));
  if (p.d_zero) {
    CK(cudaMemset(p.d_zero, 0, p.zero_elems * sizeof(float)));
    std::vector<void*> zp(p.mats.size() * (size_t)p.W, p.d_zero);
    CK(up(p.d_zero_ptrs, zp.data(), zp.size() * sizeof(void*)));
    if (p.d_zero_gmaps) {
      std::vector<uint8_t> gm(zp.size() * kTcMapBytes);
      rc = tc_encode_grad_maps(p.layers.data(), (int)p.layers.size(), p.W, zp.data(), gm.data());
      if (rc != LQSGD_OK) { g_cuda_error = "cuTensorMapEncodeTiled failed or is not available"; return rc; }
      CK(up(p.d_zero_gmaps, gm.data(), gm.size()));
    }
  }
  // Q_0
  std::vector<float> q0;
  for (size_t li = 0; li < p.mats.size(); ++li) {
    const MatHost& mt = p.mats[li];
    q0.assign((size_t)mt.m * p.RP, 0.f);
    for (int i = 0; i < mt.m; ++i)
      for (int j = 0; j < mt.r; ++j)
        q0[(size_t)i * p.RP + j] = normal_draw(cfg->seed, (uint64_t)mt.user_index, (uint64_t)i * mt.r + j);
    CK(up(p.layers[li].Q, q0.data(), q0.size() * sizeof(float)));
    CK(launch_q_transpose(p.layers[li].Q, p.layers[li].Qt, p.layers[li].Qcat, mt.m, p.RP, p.layers[li].mt, p.layers[li].kcat,
                          p.layers[li].tc, nullptr));
  }
  int o1 = 1, o2 = 1, o3 = 1;
  CK(pass_occupancy(p.RP, &o1, &o2, &o3));
  c->grid1 = (int)std::min<size_t>(p.tiles1.size(), (size_t)c->sm_count * std::max(o1, 1));
  c->grid2 = (int)p.tiles2.size();   // one CTA per tile: the hardware scheduler balances them
  c->grid3 = (int)std::min<size_t>(p.tiles3.size(), (size_t)c->sm_count * std::max(o3, 1));
  c->ptr_count = (p.mats.size() + p.vecs.size()) * (size_t)(p.W + 2);
  c->ptr_sets.assign(kPtrSets, std::vector<void*>());
  c->ptr_used.assign(kPtrSets, 0);
  c->ptr_pinned.assign(kPtrSets, 0);
  CK(cudaDeviceSynchronize());
  guard.c = nullptr;
  *ctx_out = c;
  return LQSGD_OK;
}

void lqsgd_destroy(lqsgd_ctx* ctx) { delete ctx; }

int lqsgd_set_phase_events(lqsgd_ctx* c, void* const* host_events) {
  if (!c) return LQSGD_ERR_INVALID_ARG;
  c->have_events = false;
  if (!host_events) return LQSGD_OK;
  for (int i = 0; i <= LQSGD_N_PHASES; ++i) {
    if (!host_events[i]) return LQSGD_ERR_INVALID_ARG;
    c->phase_events[i] = static_cast<cudaEvent_t>(host_events[i]);
  }
  c->have_events = true;
  return LQSGD_OK;
}

int lqsgd_test_expire_wait(lqsgd_ctx* c, int32_t pass, int32_t stage, uint32_t wait_limit) {
  if (!c || pass < 1 || pass > 4 || stage < 0 || wait_limit < 16 || wait_limit > (1u << 18)) return LQSGD_ERR_INVALID_ARG;
  c->test_wait_limit = wait_limit;
  c->test_skip_pass = pass;
  c->test_skip_stage = stage;
  return LQSGD_OK;
}

int lqsgd_check_guards(const lqsgd_ctx* c, int64_t* host_changed_words, int64_t* host_first_offset, void* cuda_stream) {
  if (!c || !host_changed_words) return LQSGD_ERR_INVALID_ARG;
  const Plan& p = c->plan;
  if (p.guards.empty()) return LQSGD_ERR_INVALID_ARG;            // created without LQSGD_FLAG_GUARD_WORDS
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CK(cudaMemsetAsync(p.d_guard_result, 0xff, 2 * sizeof(unsigned long long), st));
  CK(cudaMemsetAsync(p.d_guard_result, 0, sizeof(unsigned long long), st));
  CK(launch_guards(static_cast<char*>(c->workspace), p.d_guards, (int)p.guards.size(), kGuardPattern, p.d_guard_result, st));
  unsigned long long res[2] = {0, 0};
  CK(cudaMemcpyAsync(res, p.d_guard_result, sizeof(res), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  *host_changed_words = (int64_t)res[0];
  if (host_first_offset) *host_first_offset = res[0] ? (int64_t)res[1] : -1;
  return LQSGD_OK;
}

int lqsgd_round_timeline(const lqsgd_ctx* c, uint64_t* host_ns, int32_t* host_count, void* cuda_stream) {
  if (!c || !host_ns || !host_count) return LQSGD_ERR_INVALID_ARG;
  *host_count = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (!c->plan.resident) { CK(cudaStreamSynchronize(st)); return LQSGD_OK; }
  uint64_t tmp[kResStamps + 1] = {};
  CK(cudaMemcpyAsync(tmp, c->plan.d_rstamps, sizeof(tmp), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  const int n = (int)std::min<uint64_t>(tmp[kResStamps], (uint64_t)LQSGD_TIMELINE_MAX);
  for (int i = 0; i < n; ++i) host_ns[i] = tmp[i];
  *host_count = n;
  return LQSGD_OK;
}

int lqsgd_release_graph_tables(lqsgd_ctx* c) {
  if (!c) return LQSGD_ERR_INVALID_ARG;
  std::fill(c->ptr_pinned.begin(), c->ptr_pinned.end(), 0);
  return LQSGD_OK;
}

int lqsgd_launches_per_step(const lqsgd_ctx* ctx, int32_t* out) {
  if (!ctx || !out) return LQSGD_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  if (p.resident) { *out = 1; return LQSGD_OK; }              // the whole round is one cooperative launch
  // Orthonormalize, exchange of P, Q_w reduction, exchange of Q; then one launch per non-empty tile list
  const int pass1 = (p.tiles1.empty() ? 0 : 1) + (p.stiles1.empty() ? 0 : 1) + (p.tctiles1.empty() ? 0 : 1);
  const int pass2 = (p.tiles2.empty() ? 0 : 1) + (p.tctiles2.empty() ? 0 : 1);
  const int pass3 = (p.tiles3.empty() ? 0 : 1) + (p.stiles3.empty() ? 0 : 1) + (p.tctiles3.empty() ? 0 : 1);
  const int iters = std::max(1, ctx->cfg.power_iters);
  const int orth = (p.fbS.empty() ? 0 : 1) + (p.fbP.empty() ? 0 : 2) + (p.fbC.empty() ? 0 : 1);   // one CTA per small layer / Gram (+ Cholesky) + apply
  const int folds = (p.foldP.empty() ? 0 : 1) + (p.foldG.empty() ? 0 : 1) + (p.foldQ.empty() ? 0 : 1);
  *out = iters * ((p.mats.empty() ? 0 : orth + 2 + (p.fbQ.empty() ? 0 : 1) + folds) + pass1 + pass2) + pass3 + ((p.chV.empty() || vectors_ride(ctx)) ? 0 : 1);
  return LQSGD_OK;
}

// Checks and uploads the step's pointers and fills the kernels' table.  ghat == nullptr (only with weights): G_hat is not
// written.  Pointer table: [grads nm*W | ghat nm | weights nm | vgrads nv*W | vghat nv | vweights nv].
static int prepare_step(lqsgd_ctx* c, const float* const* grads, float* const* ghat, float* const* weights, float lr,
                        void* cuda_stream) {
  if (!c || !grads || (!ghat && !weights)) return LQSGD_ERR_INVALID_ARG;
  Plan& p = c->plan;
  const int W = p.W, nl = (int)c->shapes.size();
  const size_t nm = p.mats.size(), nv = p.vecs.size();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  std::vector<void*> ptrs(c->ptr_count);
  auto out_ptr = [&](float* const* arr, int ui, uintptr_t amask, void** slot) -> int {
    float* q = arr ? arr[ui] : nullptr;
    if (reinterpret_cast<uintptr_t>(q) & amask) return LQSGD_ERR_MISALIGNED;
    *slot = q;
    return LQSGD_OK;
  };
  for (size_t li = 0; li < nm; ++li) {
    const int ui = p.mats[li].user_index;
    const uintptr_t amask = (p.mats[li].m % 4 == 0) ? 15 : 3;
    for (int w = 0; w < W; ++w) {
      const float* g = grads[(size_t)w * nl + ui];
      if (!g) return LQSGD_ERR_INVALID_ARG;
      if (reinterpret_cast<uintptr_t>(g) & amask) return LQSGD_ERR_MISALIGNED;
      ptrs[li * W + w] = const_cast<float*>(g);
    }
    int rc = out_ptr(ghat, ui, amask, &ptrs[nm * W + li]);
    if (rc == LQSGD_OK) rc = out_ptr(weights, ui, amask, &ptrs[nm * (W + 1) + li]);
    if (rc != LQSGD_OK) return rc;
    if (!ptrs[nm * W + li] && !ptrs[nm * (W + 1) + li]) return LQSGD_ERR_INVALID_ARG;   // nowhere to put the result
  }
  const size_t vbase = nm * (W + 2);
  for (size_t vi = 0; vi < nv; ++vi) {
    const int ui = p.vecs[vi].user_index;
    for (int w = 0; w < W; ++w) {
      const float* g = grads[(size_t)w * nl + ui];
      if (!g) return LQSGD_ERR_INVALID_ARG;
      if (reinterpret_cast<uintptr_t>(g) & 3) return LQSGD_ERR_MISALIGNED;
      ptrs[vbase + vi * W + w] = const_cast<float*>(g);
    }
    int rc = out_ptr(ghat, ui, 3, &ptrs[vbase + nv * W + vi]);
    if (rc == LQSGD_OK) rc = out_ptr(weights, ui, 3, &ptrs[vbase + nv * (W + 1) + vi]);
    if (rc != LQSGD_OK) return rc;
    if (!ptrs[vbase + nv * W + vi] && !ptrs[vbase + nv * (W + 1) + vi]) return LQSGD_ERR_INVALID_ARG;
  }
  // a table already on the device?  else upload it over the slot used longest ago
  int slot = -1;
  for (int k = 0; k < kPtrSets && slot < 0; ++k)
    if (c->ptr_sets[k] == ptrs) slot = k;
  ++c->step_counter;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  CK(cudaStreamIsCapturing(st, &cap));
  if (slot < 0) {
    if (cap != cudaStreamCaptureStatusNone) return LQSGD_ERR_CAPTURE;   // a copy from this host vector cannot be replayed
    for (int k = 0; k < kPtrSets; ++k)
      if (!c->ptr_pinned[k] && (slot < 0 || c->ptr_used[k] < c->ptr_used[slot])) slot = k;
    if (slot < 0) return LQSGD_ERR_CAPTURE;                             // every table belongs to a captured graph
    // the host mirror names the slot's contents only once the copy has been accepted: after a failed copy the
    // slot matches no pointer set, so no later call can take the stale device table for its own
    c->ptr_sets[slot].clear();
    // stream-ordered after the kernels that may still read the slot; pageable source: the runtime stages it before
    // returning, so the vector may go afterwards
    CK(cudaMemcpyAsync(p.d_ptrs + (size_t)slot * c->ptr_count, ptrs.data(), ptrs.size() * sizeof(void*),
                       cudaMemcpyHostToDevice, st));
    if (p.d_gmaps) {
      // the tensor-core pass 1 reads the gradients through tensor maps: encoded once per pointer set, kept with the table
      std::vector<uint8_t> gm(nm * (size_t)W * kTcMapBytes);
      if (tc_encode_grad_maps(p.layers.data(), (int)nm, W, ptrs.data(), gm.data()) != LQSGD_OK) {
        g_cuda_error = "cuTensorMapEncodeTiled failed on a gradient tensor";
        return LQSGD_ERR_CUDA;
      }
      CK(cudaMemcpyAsync(p.d_gmaps + (size_t)slot * gm.size(), gm.data(), gm.size(), cudaMemcpyHostToDevice, st));
    }
    c->ptr_sets[slot] = ptrs;
  }
  c->ptr_used[slot] = c->step_counter;
  if (cap != cudaStreamCaptureStatusNone) c->ptr_pinned[slot] = 1;
  void** dp = p.d_ptrs + (size_t)slot * c->ptr_count;
  c->ptrs_cur = dp;
  Tables& t = c->tables;
  t.layers = p.d_layers;
  t.grads = reinterpret_cast<const float* const*>(dp);
  t.ghat = reinterpret_cast<float* const*>(dp + nm * W);
  t.weights = weights ? reinterpret_cast<float* const*>(dp + nm * (W + 1)) : nullptr;
  t.lr = lr;
  t.payload = p.d_payload;
  t.payload_stride = p.payload_stride;
  t.status = p.d_status;
  t.gmaps = p.d_gmaps ? p.d_gmaps + (size_t)slot * nm * (size_t)W * kTcMapBytes : nullptr;
  t.W = W;
  t.col_scales = (c->cfg.flags & LQSGD_FLAG_COLUMN_SCALES) ? 1 : 0;
  t.clear_status = 0;
  t.wait_limit = c->test_wait_limit;          // zero unless a test armed them for this step
  t.test_skip_pass = c->test_skip_pass;
  t.test_skip_stage = c->test_skip_stage;
  c->test_wait_limit = 0;
  c->test_skip_pass = c->test_skip_stage = 0;
  c->has_weights = weights != nullptr;
  return LQSGD_OK;
}

// The launch sequence, cut into the segments between which a multi-GPU run exchanges data.
//   0: 1-D tensors, pass 1, Orthonormalize (+ local scales of P when split)
//   1: exchange of P - fused (quantise, pack, sum, dequantise) or, when split, quantise + pack only
//   2: (split: sum over all ranks' streams + dequantise P) pass 2, Q_w (+ local scales of Q when split)
//   3: exchange of Q, as segment 1
//   4: (split: sum + dequantise Q)     5: pass 3
static int run_segment(lqsgd_ctx* c, int seg, bool split, const void* gathered, int n_streams, cudaStream_t st,
                       bool repeat = false) {
  Plan& p = c->plan;
  // a repeated power step (power_iters > 1) runs pass 1 on M itself: its "gradient" is the zero buffer
  Tables t = c->tables;
  if (repeat) { t.grads = reinterpret_cast<const float* const*>(p.d_zero_ptrs); t.gmaps = p.d_zero_gmaps; }
  const int W = p.W, RP = p.RP;
  const size_t nm = p.mats.size(), nv = p.vecs.size();
  const size_t vbase = nm * (W + 2);
  const int avg_values = (c->cfg.flags & LQSGD_FLAG_AVERAGE_VALUES) ? 1 : 0;
  const QuantTables qp{p.d_thrP, p.d_deqP, c->cfg.bits_p, avg_values}, qq{p.d_thrQ, p.d_deqQ, c->cfg.bits_q, avg_values};
  SplitExchange sx{};
  sx.pack_only = split ? 1 : 0;
  sx.n_mat = (int)nm;
  sx.scales = p.d_xscales;
  sx.ns = p.xscale_ns;
  sx.send[0] = p.d_xsend[0]; sx.send[1] = p.d_xsend[1];
  sx.region_bytes[0] = p.region_bytes[0]; sx.region_bytes[1] = p.region_bytes[1];
  sx.region_off[0] = p.region_off[0]; sx.region_off[1] = p.region_off[1];
  VectorJob vj{};
  vj.vecs = p.d_vecs; vj.chunks = p.d_chV; vj.nchunks = (int)p.chV.size(); vj.W_total = p.W_total;
  vj.vgrads = reinterpret_cast<const float* const*>(c->ptrs_cur + vbase);
  vj.vghat = reinterpret_cast<float* const*>(c->ptrs_cur + vbase + nv * W);
  vj.vweights = c->has_weights ? reinterpret_cast<float* const*>(c->ptrs_cur + vbase + nv * (W + 1)) : nullptr;
  vj.lr = t.lr;
  vj.xvec = split ? p.d_xvec : nullptr;
  vj.xvec_base = p.vec_pay_base;
  const bool ride = vectors_ride(c);     // the 1-D tensors travel as extra blocks of the exchange of P
  const bool ev = c->have_events && !split;
  // the register kernel of a pass beside its big kernel (see lqsgd_ctx::side): fork, launch it, launch the big one, join
  const bool beside = c->side != nullptr;
  cudaStream_t small = beside ? c->side : st;
  auto fork = [&]() -> cudaError_t {
    if (!beside) return cudaSuccess;
    cudaError_t e = cudaEventRecord(c->ev_fork, st);
    return e != cudaSuccess ? e : cudaStreamWaitEvent(c->side, c->ev_fork, 0);
  };
  auto forked = [&]() -> cudaError_t { return beside ? cudaEventRecord(c->ev_join, c->side) : cudaSuccess; };
  auto join = [&]() -> cudaError_t { return beside ? cudaStreamWaitEvent(st, c->ev_join, 0) : cudaSuccess; };
#define PHASE_MARK(i) do { if (ev) CK(cudaEventRecord(c->phase_events[i], st)); } while (0)
  static const char* const kSegName[6] = {"lqsgd: pass 1 + Orthonormalize", "lqsgd: exchange of P", "lqsgd: pass 2 + Q_w",
                                          "lqsgd: exchange of Q", "lqsgd: sum of Q over ranks", "lqsgd: pass 3"};
  NvtxRange nvtx(kSegName[seg >= 0 && seg <= 5 ? seg : 0]);
  switch (seg) {
    case 0:
      if (nv && !repeat) {
        if ((c->cfg.flags & LQSGD_FLAG_QUANTIZE_VECTORS) && c->cfg.bits_p != 32) {
          if (split) return LQSGD_ERR_INVALID_ARG;
          CK(launch_vectors_quant(p.d_vecs, (int)nv, reinterpret_cast<const float* const*>(c->ptrs_cur + vbase),
                                  reinterpret_cast<float* const*>(c->ptrs_cur + vbase + nv * W),
                                  c->has_weights ? reinterpret_cast<float* const*>(c->ptrs_cur + vbase + nv * (W + 1)) : nullptr,
                                  t.lr, p.d_payload, p.payload_stride, W, qp, {st, 0}));
        } else if (!ride) {
          CK(launch_vectors(vj, p.d_payload, p.payload_stride, W, {st, 0}));
        }
      }
      if (!repeat) PHASE_MARK(0);
      if (nm) {
        // the first pass-1 launch of the round zeroes the status words (see clear_status_words)
        Tables first = t, rest = t;
        first.clear_status = repeat ? 0 : (int)nm;
        rest.clear_status = 0;
        const bool reg1 = !p.tiles1.empty(), st1 = !p.stiles1.empty();
        const bool own = reg1 && !beside;      // the register kernel zeroes the words only when it runs in front
        CK(fork());
        CK(launch_pass1(RP, own ? first : rest, p.d_tiles1, (int)p.tiles1.size(), {small, c->grid1}));
        CK(forked());
        CK(launch_stream_pass1(RP, (!own && st1) ? first : rest, p.d_stiles1, (int)p.stiles1.size(),
                               {st, (int)std::min<size_t>(p.stiles1.size(), c->sm_count)}));
        CK(launch_tc_pass1(RP, (!own && !st1) ? first : rest, p.d_tctiles1, (int)p.tctiles1.size(), p.d_tcsched, p.d_tcmaps,
                           {st, p.tc_grid}));
        CK(join());
      }
      PHASE_MARK(1);
      if (nm) {
        CK(launch_fold(p.d_foldP, (int)p.foldP.size(), {st, 0}));
        CK(launch_p_orth_small(RP, t, p.d_fbS, (int)p.fbS.size(), {st, 0}));
        CK(launch_p_reduce_gram(RP, t, p.d_fbP, (int)p.fbP.size(), {st, 0}));
        CK(launch_fold(p.d_foldG, (int)p.foldG.size(), {st, 0}));
        if (RP >= kCholSplitRP) CK(launch_p_chol(RP, t, p.d_fbC, (int)p.fbC.size(), {st, 0}));
        CK(launch_p_apply(RP, t, p.d_fbP, (int)p.fbP.size(), {st, 0}));
        if (split) CK(launch_scale_reduce(RP, t, 0, p.d_xscales, (int)nm, {st, 0}));
      }
      break;
    case 1:
      if (nm) CK(launch_exchange(RP, 0, t, qp, p.d_chP, (int)p.chP.size(), sx, (ride && !repeat) ? &vj : nullptr, {st, 0}));
      PHASE_MARK(2);
      break;
    case 2:
      if (nm) {
        if (split) CK(launch_sum_dequant(RP, 0, t, qp, p.d_chP, (int)p.chP.size(), sx, static_cast<const uint8_t*>(gathered), n_streams, {st, 0}));
        const bool beside2 = beside && !p.tctiles2.empty();       // (staged layers have no big kernel in this pass)
        if (beside2) CK(fork());
        CK(launch_pass2(RP, t, p.d_tiles2, (int)p.tiles2.size(), {beside2 ? small : st, c->grid2}));
        if (beside2) CK(forked());
        CK(launch_tc_pass2(RP, t, p.d_tctiles2, (int)p.tctiles2.size(), p.d_tcmaps,
                           {st, (int)std::min<size_t>(p.tctiles2.size(), c->sm_count)}));
        if (beside2) CK(join());
      }
      PHASE_MARK(3);
      if (nm) {
        CK(launch_fold(p.d_foldQ, (int)p.foldQ.size(), {st, 0}));
        CK(launch_q_reduce(RP, t, p.d_fbQ, (int)p.fbQ.size(), {st, 0}));
        if (split) CK(launch_scale_reduce(RP, t, 1, p.d_xscales, (int)nm, {st, 0}));
      }
      break;
    case 3:
      if (nm) CK(launch_exchange(RP, 1, t, qq, p.d_chQ, (int)p.chQ.size(), sx, nullptr, {st, 0}));
      PHASE_MARK(4);
      break;
    case 4:
      if (nm && split) CK(launch_sum_dequant(RP, 1, t, qq, p.d_chQ, (int)p.chQ.size(), sx, static_cast<const uint8_t*>(gathered), n_streams, {st, 0}));
      break;
    case 5:
      if (nm) {
        const bool beside3 = beside && !p.tiles3.empty();
        if (beside3) CK(fork());
        CK(launch_pass3(RP, t, p.d_tiles3, (int)p.tiles3.size(), {beside3 ? small : st, c->grid3}));
        if (beside3) CK(forked());
        CK(launch_stream_pass3(RP, t, p.d_stiles3, (int)p.stiles3.size(), {st, (int)std::min<size_t>(p.stiles3.size(), c->sm_count)}));
        CK(launch_tc_pass3(RP, t, p.d_tctiles3, (int)p.tctiles3.size(), p.d_tcsched + 4, p.d_tcmaps, {st, p.tc_grid}));
        if (beside3) CK(join());
      }
      if (split && nv) CK(launch_vectors_finish(vj, {st, 0}));     // the shares were summed over the ranks meanwhile
      PHASE_MARK(5);
      break;
    default: return LQSGD_ERR_INVALID_ARG;
  }
#undef PHASE_MARK
  return LQSGD_OK;
}

// The whole round as one cooperative launch (sets that fit the SMs' shared memory; see lqsgd_resident.cu).
static int run_resident(lqsgd_ctx* c, cudaStream_t st) {
  Plan& p = c->plan;
  const int W = p.W;
  const size_t nm = p.mats.size(), nv = p.vecs.size();
  const size_t vbase = nm * (W + 2);
  const int avg_values = (c->cfg.flags & LQSGD_FLAG_AVERAGE_VALUES) ? 1 : 0;
  Tables t = c->tables;
  t.clear_status = (int)nm;
  ResidentArgs a{};
  a.tiles = p.d_rtiles; a.cta_begin = p.d_rbegin;
  a.fbS = p.d_fbS; a.nfbS = (int)p.fbS.size();
  a.fbP = p.d_fbP; a.nfbP = (int)p.fbP.size();
  a.fbQ = p.d_fbQ; a.nfbQ = (int)p.fbQ.size();
  a.chP = p.d_chP; a.nchP = (int)p.chP.size();
  a.chQ = p.d_chQ; a.nchQ = (int)p.chQ.size();
  a.qp = QuantTables{p.d_thrP, p.d_deqP, c->cfg.bits_p, avg_values};
  a.qq = QuantTables{p.d_thrQ, p.d_deqQ, c->cfg.bits_q, avg_values};
  a.vj.vecs = p.d_vecs; a.vj.chunks = p.d_chV; a.vj.nchunks = (int)p.chV.size(); a.vj.W_total = p.W_total;
  a.vj.vgrads = reinterpret_cast<const float* const*>(c->ptrs_cur + vbase);
  a.vj.vghat = reinterpret_cast<float* const*>(c->ptrs_cur + vbase + nv * W);
  a.vj.vweights = c->has_weights ? reinterpret_cast<float* const*>(c->ptrs_cur + vbase + nv * (W + 1)) : nullptr;
  a.vj.lr = t.lr;
  a.sync = p.d_rsync;
  a.stamps = p.d_rstamps;
  // phase events: one kernel, so the round's time shows as its first phase and the others as empty
  NvtxRange nvtx("lqsgd: round in one launch");
  if (c->have_events) CK(cudaEventRecord(c->phase_events[0], st));
  CK(launch_resident(p.RP, t, a, p.res_grid, p.res_smem, st));
  if (c->have_events)
    for (int i = 1; i <= LQSGD_N_PHASES; ++i) CK(cudaEventRecord(c->phase_events[i], st));
  c->have_events = false;
  return LQSGD_OK;
}

static int step_impl(lqsgd_ctx* c, const float* const* grads, float* const* ghat, float* const* weights, float lr,
                     void* cuda_stream) {
  int rc = prepare_step(c, grads, ghat, weights, lr, cuda_stream);
  if (rc != LQSGD_OK) return rc;
  if (c->plan.W_total != c->plan.W) return LQSGD_ERR_INVALID_ARG;   // workers elsewhere: use the lqsgd_round_* calls
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (c->plan.resident) return run_resident(c, st);
  const int iters = std::max(1, c->cfg.power_iters);
  for (int it = 0; it < iters; ++it)
    for (int seg = 0; seg <= 4; ++seg) {
      rc = run_segment(c, seg, false, nullptr, 0, st, it > 0);
      if (rc != LQSGD_OK) return rc;
    }
  rc = run_segment(c, 5, false, nullptr, 0, st);
  if (rc != LQSGD_OK) return rc;
  c->have_events = false;
  return LQSGD_OK;
}

int lqsgd_step(lqsgd_ctx* c, const float* const* grads, float* const* ghat, void* cuda_stream) {
  if (!ghat) return LQSGD_ERR_INVALID_ARG;
  return step_impl(c, grads, ghat, nullptr, 0.f, cuda_stream);
}

int lqsgd_step_update(lqsgd_ctx* c, const float* const* grads, float* const* ghat, float* const* weights, float lr,
                      void* cuda_stream) {
  if (!weights) return LQSGD_ERR_INVALID_ARG;
  return step_impl(c, grads, ghat, weights, lr, cuda_stream);
}

// ---- the same round in pieces, for workers spread over several GPUs (see include/lqsgd.h)
int lqsgd_round_begin(lqsgd_ctx* c, const float* const* grads, float* const* ghat, float* const* weights, float lr,
                      void* cuda_stream) {
  const int rc = prepare_step(c, grads, ghat, weights, lr, cuda_stream);
  if (rc != LQSGD_OK) return rc;
  if (c->cfg.power_iters > 1) return LQSGD_ERR_INVALID_ARG;
  if ((c->cfg.flags & LQSGD_FLAG_QUANTIZE_VECTORS) && c->cfg.bits_p != 32 && !c->plan.vecs.empty()) return LQSGD_ERR_INVALID_ARG;
  c->round_stage = 0;
  const int rs = run_segment(c, 0, true, nullptr, 0, static_cast<cudaStream_t>(cuda_stream));
  if (rs == LQSGD_OK) c->round_stage = 1;
  return rs;
}

int lqsgd_round_pack(lqsgd_ctx* c, int32_t which, void* cuda_stream) {
  if (!c || (which != 0 && which != 1)) return LQSGD_ERR_INVALID_ARG;
  if (c->round_stage != (which ? 3 : 1)) return LQSGD_ERR_INVALID_ARG;       // out of order
  const int rs = run_segment(c, which ? 3 : 1, true, nullptr, 0, static_cast<cudaStream_t>(cuda_stream));
  if (rs == LQSGD_OK) c->round_stage += 1;
  return rs;
}

int lqsgd_round_reduce(lqsgd_ctx* c, int32_t which, const void* dev_gathered, int32_t n_ranks, void* cuda_stream) {
  if (!c || !dev_gathered || (which != 0 && which != 1)) return LQSGD_ERR_INVALID_ARG;
  if (c->round_stage != (which ? 4 : 2)) return LQSGD_ERR_INVALID_ARG;       // out of order
  if (n_ranks < 1 || n_ranks * c->plan.W != c->plan.W_total) return LQSGD_ERR_INVALID_ARG;
  const int rs = run_segment(c, which ? 4 : 2, true, dev_gathered, c->plan.W_total, static_cast<cudaStream_t>(cuda_stream));
  if (rs == LQSGD_OK) c->round_stage += 1;
  return rs;
}

int lqsgd_round_end(lqsgd_ctx* c, void* cuda_stream) {
  if (!c || c->round_stage != 5) return LQSGD_ERR_INVALID_ARG;
  const int rs = run_segment(c, 5, true, nullptr, 0, static_cast<cudaStream_t>(cuda_stream));
  c->round_stage = 0;
  return rs;
}

int lqsgd_exchange_view(const lqsgd_ctx* c, int32_t which, void** dev_ptr, size_t* bytes) {
  if (!c || !dev_ptr || !bytes) return LQSGD_ERR_INVALID_ARG;
  const Plan& p = c->plan;
  switch (which) {
    case LQSGD_XCHG_SCALES_P: *dev_ptr = p.d_xscales; *bytes = 4 * p.mats.size() * p.xscale_ns; break;
    case LQSGD_XCHG_SCALES_Q: *dev_ptr = p.d_xscales + p.mats.size() * p.xscale_ns; *bytes = 4 * p.mats.size() * p.xscale_ns; break;
    case LQSGD_XCHG_VECTORS: *dev_ptr = p.d_xvec; *bytes = 4 * p.vec_elems; break;
    case LQSGD_XCHG_STREAMS_P: *dev_ptr = p.d_xsend[0]; *bytes = (size_t)p.W * p.region_bytes[0]; break;
    case LQSGD_XCHG_STREAMS_Q: *dev_ptr = p.d_xsend[1]; *bytes = (size_t)p.W * p.region_bytes[1]; break;
    default: return LQSGD_ERR_OUT_OF_RANGE;
  }
  return LQSGD_OK;
}

int lqsgd_step_host(lqsgd_ctx* c, const float* const* host_grads, float* const* host_ghat,
                    void* host_payload, void* cuda_stream) {
  if (!c || !host_grads || !host_ghat) return LQSGD_ERR_INVALID_ARG;
  Plan& p = c->plan;
  if (!p.d_stage_g) return LQSGD_ERR_NO_STAGING;
  const int W = p.W, nl = (int)c->shapes.size();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  std::vector<const float*> dg((size_t)W * nl);
  std::vector<float*> dh(nl);
  // Copies of tensors that follow one another both in the caller's memory and in the staging area are merged
  // into one: a gradient set kept in one host buffer per worker goes up in a few large copies instead of one
  // per tensor (most tensors of a network are a few hundred bytes of batch-norm parameters).
  // (Neighbours in address space need not belong to one allocation: if the runtime refuses a merged copy, its
  // pieces go one by one.)
  struct Piece { char* dst; const char* src; size_t bytes; };
  struct Run { std::vector<Piece> pieces; size_t bytes = 0; };
  auto flush = [&](Run& r, cudaMemcpyKind kind) -> cudaError_t {
    cudaError_t e = cudaSuccess;
    if (!r.pieces.empty()) {
      e = cudaMemcpyAsync(r.pieces[0].dst, r.pieces[0].src, r.bytes, kind, st);
      if (e != cudaSuccess && r.pieces.size() > 1) {
        (void)cudaGetLastError();                                  // not sticky: clear it and copy piece by piece
        e = cudaSuccess;
        for (const Piece& pc : r.pieces)
          if (e == cudaSuccess) e = cudaMemcpyAsync(pc.dst, pc.src, pc.bytes, kind, st);
      }
    }
    r.pieces.clear();
    r.bytes = 0;
    return e;
  };
  auto add = [&](Run& r, void* dst, const void* src, size_t bytes, cudaMemcpyKind kind) -> cudaError_t {
    cudaError_t e = cudaSuccess;
    if (!r.pieces.empty() && !(r.pieces[0].dst + r.bytes == dst && r.pieces[0].src + r.bytes == src)) e = flush(r, kind);
    r.pieces.push_back(Piece{static_cast<char*>(dst), static_cast<const char*>(src), bytes});
    r.bytes += bytes;
    return e;
  };
  for (int l = 0; l < nl; ++l) {
    if (!host_ghat[l]) return LQSGD_ERR_INVALID_ARG;
    dh[l] = p.d_stage_ghat + p.elem_off[l];
    for (int w = 0; w < W; ++w)
      if (!host_grads[(size_t)w * nl + l]) return LQSGD_ERR_INVALID_ARG;
  }
  Run run;
  for (int w = 0; w < W; ++w)
    for (int l = 0; l < nl; ++l) {
      const size_t bytes = 4 * (size_t)c->shapes[l].rows * c->shapes[l].cols;
      float* dst = p.d_stage_g + (size_t)w * p.elems_total + p.elem_off[l];
      CK(add(run, dst, host_grads[(size_t)w * nl + l], bytes, cudaMemcpyHostToDevice));
      dg[(size_t)w * nl + l] = dst;
    }
  CK(flush(run, cudaMemcpyHostToDevice));
  const int rc = lqsgd_step(c, dg.data(), dh.data(), cuda_stream);
  if (rc != LQSGD_OK) return rc;
  for (int l = 0; l < nl; ++l) {
    const size_t bytes = 4 * (size_t)c->shapes[l].rows * c->shapes[l].cols;
    CK(add(run, host_ghat[l], dh[l], bytes, cudaMemcpyDeviceToHost));
  }
  CK(flush(run, cudaMemcpyDeviceToHost));
  if (host_payload) {
    CK(cudaMemcpy2DAsync(host_payload, p.payload_bytes, p.d_payload, p.payload_stride, p.payload_bytes, W,
                         cudaMemcpyDeviceToHost, st));
  }
  CK(cudaStreamSynchronize(st));
  return LQSGD_OK;
}

int lqsgd_payload_bytes(const lqsgd_ctx* c, size_t* out) {
  if (!c || !out) return LQSGD_ERR_INVALID_ARG;
  *out = c->plan.payload_bytes;
  return LQSGD_OK;
}

int lqsgd_payload(const lqsgd_ctx* c, int32_t worker, const void** dev_ptr, size_t* bytes) {
  if (!c || !dev_ptr || !bytes) return LQSGD_ERR_INVALID_ARG;
  if (worker < 0 || worker >= c->plan.W) return LQSGD_ERR_OUT_OF_RANGE;
  *dev_ptr = c->plan.d_payload + (size_t)worker * c->plan.payload_stride;
  *bytes = c->plan.payload_bytes;
  return LQSGD_OK;
}

int lqsgd_payload_layout(const lqsgd_ctx* c, int32_t layer, lqsgd_layer_layout* out) {
  if (!c || !out) return LQSGD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= (int)c->shapes.size()) return LQSGD_ERR_OUT_OF_RANGE;
  *out = c->plan.layout[layer];
  return LQSGD_OK;
}

// Locates a piece of state: base pointer, rows, dense row bytes, stored row pitch in bytes.
static int locate_state(const lqsgd_ctx* c, int which, int layer, int worker, char** base, size_t* rows,
                        size_t* row_bytes, size_t* pitch) {
  if (layer < 0 || layer >= (int)c->shapes.size()) return LQSGD_ERR_OUT_OF_RANGE;
  const Plan& p = c->plan;
  int li = -1;
  for (size_t i = 0; i < p.mats.size(); ++i)
    if (p.mats[i].user_index == layer) li = (int)i;
  if (li < 0) return LQSGD_ERR_OUT_OF_RANGE;          // 1-D tensors carry no state
  const LayerDev& L = p.layers[li];
  const size_t n = L.n, m = L.m, r = L.r, RP = p.RP, W = p.W;
  const bool per_worker = which == LQSGD_STATE_E || which == LQSGD_STATE_P_RAW || which == LQSGD_STATE_P ||
                          which == LQSGD_STATE_Q_W || which == LQSGD_STATE_CODES_P || which == LQSGD_STATE_CODES_Q;
  if (per_worker && (worker < 0 || worker >= (int)W)) return LQSGD_ERR_OUT_OF_RANGE;
  const size_t w = per_worker ? worker : 0;
  switch (which) {
    case LQSGD_STATE_E: *base = (char*)(L.E + w * n * m); *rows = 1; *row_bytes = *pitch = 4 * n * m; break;
    case LQSGD_STATE_Q: *base = (char*)L.Q; *rows = m; *row_bytes = 4 * r; *pitch = 4 * RP; break;
    case LQSGD_STATE_P_RAW: *base = (char*)(L.Praw + w * n * RP); *rows = n; *row_bytes = 4 * r; *pitch = 4 * RP; break;
    case LQSGD_STATE_P: *base = (char*)(L.P + w * n * RP); *rows = n; *row_bytes = 4 * r; *pitch = 4 * RP; break;
    case LQSGD_STATE_P_BAR: *base = (char*)L.Pbar; *rows = n; *row_bytes = 4 * r; *pitch = 4 * RP; break;
    case LQSGD_STATE_Q_W: *base = (char*)(L.Qw + w * m * RP); *rows = m; *row_bytes = 4 * r; *pitch = 4 * RP; break;
    // codes are not kept unpacked: base = the worker's packed stream, rows = number of codes (see lqsgd_get_state)
    case LQSGD_STATE_CODES_P: if (c->cfg.bits_p == 32) return LQSGD_ERR_OUT_OF_RANGE; *base = (char*)(p.d_payload + w * p.payload_stride + L.pay_p_off); *rows = n * r; *row_bytes = *pitch = 1; break;
    case LQSGD_STATE_CODES_Q: if (c->cfg.bits_q == 32) return LQSGD_ERR_OUT_OF_RANGE; *base = (char*)(p.d_payload + w * p.payload_stride + L.pay_q_off); *rows = m * r; *row_bytes = *pitch = 1; break;
    case LQSGD_STATE_SCALES:
      *base = (char*)L.scales;
      if (c->cfg.flags & LQSGD_FLAG_COLUMN_SCALES) { *rows = 2; *row_bytes = 4 * r; *pitch = 4 * RP; }
      else { *rows = 1; *row_bytes = *pitch = 8; }
      break;
    default: return LQSGD_ERR_OUT_OF_RANGE;
  }
  return LQSGD_OK;
}

int lqsgd_get_state(const lqsgd_ctx* c, int32_t which, int32_t layer, int32_t worker, void* dev_dst,
                    void* cuda_stream) {
  if (!c || !dev_dst) return LQSGD_ERR_INVALID_ARG;
  char* base; size_t rows, rb, pitch;
  const int rc = locate_state(c, which, layer, worker, &base, &rows, &rb, &pitch);
  if (rc != LQSGD_OK) return rc;
  if (which == LQSGD_STATE_CODES_P || which == LQSGD_STATE_CODES_Q) {   // unpacked on demand from the payload
    CK(launch_unpack_codes(reinterpret_cast<const uint8_t*>(base), (int)rows,
                           which == LQSGD_STATE_CODES_P ? c->cfg.bits_p : c->cfg.bits_q, static_cast<uint8_t*>(dev_dst),
                           static_cast<cudaStream_t>(cuda_stream)));
    return LQSGD_OK;
  }
  CK(cudaMemcpy2DAsync(dev_dst, rb, base, pitch, rb, rows, cudaMemcpyDeviceToDevice,
                       static_cast<cudaStream_t>(cuda_stream)));
  return LQSGD_OK;
}

int lqsgd_set_state(lqsgd_ctx* c, int32_t which, int32_t layer, int32_t worker, const void* dev_src,
                    void* cuda_stream) {
  if (!c || !dev_src) return LQSGD_ERR_INVALID_ARG;
  if (which != LQSGD_STATE_E && which != LQSGD_STATE_Q) return LQSGD_ERR_OUT_OF_RANGE;
  char* base; size_t rows, rb, pitch;
  const int rc = locate_state(c, which, layer, worker, &base, &rows, &rb, &pitch);
  if (rc != LQSGD_OK) return rc;
  CK(cudaMemcpy2DAsync(base, pitch, dev_src, rb, rb, rows, cudaMemcpyDeviceToDevice,
                       static_cast<cudaStream_t>(cuda_stream)));
  if (which == LQSGD_STATE_Q) {
    for (const LayerDev& L : c->plan.layers)
      if (L.user_index == layer)
        CK(launch_q_transpose(L.Q, L.Qt, L.Qcat, L.m, c->plan.RP, L.mt, L.kcat, L.tc, static_cast<cudaStream_t>(cuda_stream)));
  }
  return LQSGD_OK;
}

int lqsgd_status(const lqsgd_ctx* c, uint32_t* host_flags, void* cuda_stream) {
  if (!c || !host_flags) return LQSGD_ERR_INVALID_ARG;
  const Plan& p = c->plan;
  for (size_t i = 0; i < c->shapes.size(); ++i) host_flags[i] = 0;
  std::vector<uint32_t> tmp(p.mats.size());
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (!tmp.empty()) {
    CK(cudaMemcpyAsync(tmp.data(), p.d_status, tmp.size() * sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
  }
  CK(cudaStreamSynchronize(st));
  for (size_t i = 0; i < p.mats.size(); ++i) host_flags[p.mats[i].user_index] = tmp[i];
  return LQSGD_OK;
}

int lqsgd_step_stats(const lqsgd_ctx* c, int32_t layer, lqsgd_layer_stats* out, void* cuda_stream) {
  if (!c || !out) return LQSGD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= (int)c->shapes.size()) return LQSGD_ERR_OUT_OF_RANGE;
  const Plan& p = c->plan;
  std::memset(out, 0, sizeof(*out));
  const lqsgd_layer_layout& lay = p.layout[layer];
  const bool cs = (c->cfg.flags & LQSGD_FLAG_COLUMN_SCALES) != 0;
  if (!lay.is_matrix) {
    const bool quantised = (c->cfg.flags & LQSGD_FLAG_QUANTIZE_VECTORS) && c->cfg.bits_p != 32;
    out->payload_bytes = lay.vec_bytes + (quantised ? 4 : 0);        // its scale travels too
    return LQSGD_OK;
  }
  out->payload_bytes = (cs ? 8 * (uint64_t)lay.rank_eff : 8) + lay.p_bytes + lay.q_bytes;
  int li = -1;
  for (size_t i = 0; i < p.mats.size(); ++i)
    if (p.mats[i].user_index == layer) li = (int)i;
  if (li < 0) return LQSGD_ERR_OUT_OF_RANGE;
  const MatHost& mh = p.mats[li];
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const unsigned long long init[4] = {0ull, 0ull, ~0ull, 0ull};
  CK(cudaMemcpyAsync(p.d_stats, init, sizeof(init), cudaMemcpyHostToDevice, st));
  StatsArgs a{};
  a.layers = p.d_layers + li;
  a.thr_p = p.d_thrP;
  a.thr_q = p.d_thrQ;
  a.nthr_p = c->cfg.bits_p == 32 ? 0 : (1 << (c->cfg.bits_p - 1)) - 1;
  a.nthr_q = c->cfg.bits_q == 32 ? 0 : (1 << (c->cfg.bits_q - 1)) - 1;
  a.RP = p.RP;
  a.W = p.W;
  a.column_scales = cs ? 1 : 0;
  a.out = p.d_stats;
  CK(launch_stats(a, 1, st));
  unsigned long long res[4];
  float sc[2 * kMaxRank];
  uint32_t status = 0;
  const int ns = cs ? 2 * p.RP : 2;
  CK(cudaMemcpyAsync(res, p.d_stats, sizeof(res), cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(sc, p.layers[li].scales, ns * sizeof(float), cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(&status, p.d_status + li, sizeof(status), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  out->status = status;
  out->rank_eff = mh.r;
  if (cs) {
    for (int j = 0; j < mh.r; ++j) {
      out->scale_p = std::max(out->scale_p, sc[j]);
      out->scale_q = std::max(out->scale_q, sc[p.RP + j]);
    }
  } else {
    out->scale_p = sc[0];
    out->scale_q = sc[1];
  }
  const uint32_t ratio_bits = (uint32_t)(res[2] & 0xffffffffull);
  std::memcpy(&out->pivot_ratio, &ratio_bits, 4);
  if (ratio_bits == 0xffffffffu) out->pivot_ratio = 0.f;
  out->codes_p = c->cfg.bits_p == 32 ? 0 : (uint64_t)p.W * mh.n * mh.r;
  out->codes_q = c->cfg.bits_q == 32 ? 0 : (uint64_t)p.W * mh.m * mh.r;
  out->near_p = res[0];
  out->near_q = res[1];
  return LQSGD_OK;
}

}  // extern "C"

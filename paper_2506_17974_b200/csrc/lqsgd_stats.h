// Arguments of the statistics kernel (lqsgd_stats.cu), shared with the host side (lqsgd_api.cu).
// Internal to the library.
#pragma once
#include "lqsgd_dev.h"

namespace lqsgd {

struct StatsArgs {
  const LayerDev* layers;
  const float* thr_p;        // ascending thresholds, nthr_p entries (0 with bits 32)
  const float* thr_q;
  int nthr_p, nthr_q;
  int RP, W;
  int column_scales;
  unsigned long long* out;   // [n_mat][4]: near P, near Q, pivot ratio (float bits, low word), unused
};

// Adds to out[layer][0..1] and lowers out[layer][2]; the caller sets out to {0, 0, all ones, 0} first.
cudaError_t launch_stats(const StatsArgs& a, int n_mat, cudaStream_t st);

}  // namespace lqsgd

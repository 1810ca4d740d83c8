// fathom_plan_layer_budgets: the greedy per-layer plan (Sec. 3.4 "Per-layer budgets").  Host code only: it runs
// once per deployment on a table of measured errors, not in the decode step.
//
// Budgets come from an ascending list of levels (the paper's range is 24 .. 128 bits) at a target mean.  Every layer
// starts at the lowest level; each step raises one layer by one level, choosing the layer whose error falls most per
// added bit (ties to the lower layer); a step is taken only while the summed budgets stay within target_mean * L.
#include "fathom_common.cuh"

#include <vector>

extern "C" int fathom_plan_layer_budgets(const double* err, int n_layers, int n_levels, const int* levels, double target_mean,
                                         int* level_index) {
  if (!err || !levels || !level_index || n_layers < 1 || n_levels < 1) return FATHOM_ERR_INVALID_ARG;
  if (levels[0] < 0) return FATHOM_ERR_INVALID_ARG;
  for (int i = 1; i < n_levels; ++i)
    if (levels[i] <= levels[i - 1]) return FATHOM_ERR_INVALID_ARG;
  for (long long e = 0; e < (long long)n_layers * n_levels; ++e)
    if (!(err[e] == err[e])) return FATHOM_ERR_INVALID_ARG;   // NaN has no order
  // slope[l] = error drop per bit of layer l's next level; refreshed only for the layer that moved
  std::vector<double> slope(n_layers);
  std::vector<int> bits_next(n_layers);
  auto refresh = [&](int l) {
    const int i = level_index[l];
    if (i + 1 >= n_levels) { bits_next[l] = -1; return; }
    bits_next[l] = levels[i + 1] - levels[i];
    slope[l] = (err[(size_t)l * n_levels + i] - err[(size_t)l * n_levels + i + 1]) / (double)bits_next[l];
  };
  for (int l = 0; l < n_layers; ++l) { level_index[l] = 0; refresh(l); }
  long long spent = (long long)n_layers * levels[0];
  const double cap = target_mean * (double)n_layers;
  for (;;) {
    int pick = -1;
    for (int l = 0; l < n_layers; ++l) {
      if (bits_next[l] < 0 || (double)(spent + bits_next[l]) > cap) continue;
      if (pick < 0 || slope[l] > slope[pick]) pick = l;
    }
    if (pick < 0) break;
    spent += bits_next[pick];
    ++level_index[pick];
    refresh(pick);
  }
  return FATHOM_OK;
}

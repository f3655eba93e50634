// Host helper: the structural routing configuration Omega* = L* x G* from
// leave-one-in contributions (section "Structural Pruning"): positive
// contributions are normalised into weights w_i = max(s_i, 0) / sum_j max(s_j, 0),
// the K_L layers and K_G KV-head groups of highest weight are kept (ties: lower
// index first), and a route (l, g) exposes the resources iff both are kept.
// No device work.
#include <algorithm>
#include <numeric>
#include <vector>

#include "common.cuh"

namespace {

// indices of the k largest weights, ties broken by lower index; returns their summed weight
double top_k(const double* s, int n, int k, std::vector<int>& keep) {
  std::vector<double> w(n);
  double tot = 0.0;
  for (int i = 0; i < n; ++i) { w[i] = s[i] > 0.0 ? s[i] : 0.0; tot += w[i]; }
  if (tot > 0.0) for (double& x : w) x /= tot;
  std::vector<int> order(n);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return w[a] > w[b]; });
  keep.assign(order.begin(), order.begin() + k);
  double cc = 0.0;
  for (int i : keep) cc += w[i];
  return cc;
}

}  // namespace

extern "C" RECACHE_API recache_status recache_build_routes(const double* s_layers, int32_t n_layers,
                                                           const double* s_groups, int32_t n_groups, int32_t k_layers,
                                                           int32_t k_groups, uint8_t* omega, double* cc_layers,
                                                           double* cc_groups, double* rho) {
  if (!s_layers || !s_groups || !omega || n_layers <= 0 || n_groups <= 0) return RECACHE_EINVAL;
  if (k_layers < 0 || k_layers > n_layers || k_groups < 0 || k_groups > n_groups) return RECACHE_ESHAPE;
  std::vector<int> kl, kg;
  const double ccl = top_k(s_layers, n_layers, k_layers, kl);
  const double ccg = top_k(s_groups, n_groups, k_groups, kg);
  std::fill(omega, omega + (size_t)n_layers * n_groups, (uint8_t)0);
  for (int l : kl)
    for (int g : kg) omega[(size_t)l * n_groups + g] = 1;
  if (cc_layers) *cc_layers = ccl;
  if (cc_groups) *cc_groups = ccg;
  if (rho) *rho = 1.0 - ((double)k_layers * k_groups) / ((double)n_layers * n_groups);
  return RECACHE_OK;
}

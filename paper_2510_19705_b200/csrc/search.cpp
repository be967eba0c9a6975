// Expected latency of a hierarchy (Theorem 3.2) and the search for its parameters T (Section 4),
// host side.  gamma(alpha, T_in, T_out), for which the paper gives no formula, is the expected
// number of draft/verify rounds until the yields sum to T_out when acceptances are IID with rate
// alpha and a round yields k tokens with probability alpha^(k-1) (1 - alpha), k <= T_in, or
// T_in + 1 with probability alpha^T_in.
#include <math.h>
#include <vector>

#include "../../include/hsd.h"

namespace {

double gamma_rounds(double alpha, int t_in, int t_out) {
  std::vector<double> prob(t_in + 2, 0.0), g(t_out + t_in + 2, 0.0);
  for (int k = 1; k <= t_in; ++k) prob[k] = pow(alpha, k - 1) * (1.0 - alpha);
  prob[t_in + 1] = pow(alpha, t_in);
  for (int c = t_out - 1; c >= 0; --c) {
    double v = 1.0;
    for (int k = 1; k <= t_in + 1; ++k) v += prob[k] * g[c + k];
    g[c] = v;
  }
  return g[0];
}

double top_multiplier(double alpha, int T) {
  if (alpha >= 1.0) return 1.0 / (T + 1);
  return (1.0 - alpha) / (1.0 - pow(alpha, T + 1));
}

double latency(const double *c, const double *a, int K, const int32_t *T) {
  if (K == 0) return c[0];
  double cost = T[0] * c[0];
  for (int k = 1; k < K; ++k) cost = gamma_rounds(a[k - 1], T[k - 1], T[k]) * (cost + c[k]);
  return top_multiplier(a[K - 1], T[K - 1]) * (cost + c[K]);
}

}  // namespace

extern "C" {

int hsd_expected_latency(const double *costs, const double *alphas, int n_levels, const int32_t *T, double *out) {
  if (!costs || !out || n_levels < 1 || n_levels > 16) return HSD_E_INVALID_ARG;
  if (n_levels > 1 && (!alphas || !T)) return HSD_E_INVALID_ARG;
  for (int i = 0; i + 1 < n_levels; ++i)
    if (T[i] < 1 || alphas[i] < 0.0 || alphas[i] > 1.0) return HSD_E_INVALID_ARG;
  *out = latency(costs, alphas, n_levels - 1, T);
  return HSD_OK;
}

int hsd_search_T(const double *costs, const double *alphas, int n_levels, int T_max, int monotone, int32_t *out_T,
                 double *out_latency) {
  if (!costs || n_levels < 1 || n_levels > 8 || T_max < 1 || T_max > 64) return HSD_E_INVALID_ARG;
  const int K = n_levels - 1;
  if (K > 0 && (!alphas || !out_T)) return HSD_E_INVALID_ARG;
  for (int i = 0; i < K; ++i)
    if (alphas[i] < 0.0 || alphas[i] > 1.0) return HSD_E_INVALID_ARG;
  if (K == 0) {
    if (out_latency) *out_latency = costs[0];
    return HSD_OK;
  }
  std::vector<int32_t> T(K, 1), best(K, 1);
  double best_l = -1.0;
  for (;;) {
    bool ok = true;
    if (monotone)
      for (int k = 1; k < K; ++k) ok = ok && T[k] >= T[k - 1];
    if (ok) {
      double l = latency(costs, alphas, K, T.data());
      if (best_l < 0.0 || l < best_l - 1e-15) { best_l = l; best = T; }
    }
    int k = K - 1;                      // odometer, last parameter fastest (lexicographic order)
    while (k >= 0 && T[k] == T_max) T[k--] = 1;
    if (k < 0) break;
    T[k]++;
  }
  for (int k = 0; k < K; ++k) out_T[k] = best[k];
  if (out_latency) *out_latency = best_l;
  return HSD_OK;
}

}  // extern "C"

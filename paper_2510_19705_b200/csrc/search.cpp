// Expected latency of a hierarchy (Theorem 3.2), the search for its parameters T and the search for
// the hierarchy itself (Section 4, Corollary 4.1), host side.  gamma(alpha, T_in, T_out), for which the paper gives no formula, is the expected
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

int hsd_expected_latency_literal(const double *costs, const double *alphas, int n_levels, const int32_t *T, double *out) {
  if (!costs || !out || n_levels < 1 || n_levels > 16) return HSD_E_INVALID_ARG;
  if (n_levels > 1 && (!alphas || !T)) return HSD_E_INVALID_ARG;
  const int K = n_levels - 1;
  long long span = 2;
  for (int i = 0; i < K; ++i) {
    if (T[i] < 1 || T[i] > 4096 || alphas[i] < 0.0 || alphas[i] > 1.0) return HSD_E_INVALID_ARG;
    span += T[i];
  }
  if (K == 0) { *out = costs[0]; return HSD_OK; }
  // dist[t]: probability that the level below returns t tokens; yld[y]: probability that a round yields y
  std::vector<double> dist((size_t)span + 1, 0.0), yld, mass, next;
  dist[T[0]] = 1.0;
  double cost = T[0] * costs[0];
  for (int k = 1; k <= K; ++k) {
    const double a = alphas[k - 1];
    yld.assign((size_t)span + 2, 0.0);
    for (size_t t = 1; t < dist.size(); ++t) {
      if (dist[t] == 0.0) continue;
      double aj = 1.0;                                  // a^j
      for (size_t j = 0; j < t; ++j) { yld[j + 1] += dist[t] * aj * (1.0 - a); aj *= a; }
      yld[t + 1] += dist[t] * aj;
    }
    if (k == K) {
      double mean = 0.0;
      for (size_t y = 1; y < yld.size(); ++y) mean += (double)y * yld[y];
      *out = (cost + costs[K]) / mean;
      return HSD_OK;
    }
    const int need = T[k];
    mass.assign((size_t)need + yld.size(), 0.0);        // mass[c]: probability of holding c tokens (c < need: before a round)
    mass[0] = 1.0;
    double rounds = 0.0;
    for (int c = 0; c < need; ++c) {
      const double m = mass[c];
      if (m == 0.0) continue;
      rounds += m;
      for (size_t y = 1; y < yld.size(); ++y) mass[c + y] += m * yld[y];
    }
    cost = rounds * (cost + costs[k]);
    next.assign((size_t)span + 1, 0.0);
    for (size_t c = need; c < mass.size() && c < next.size(); ++c) next[c] = mass[c];
    dist.swap(next);
  }
  return HSD_E_INVALID_ARG;
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

// Latency-optimal hierarchy (Section 4.2).  The paper reduces the choice of (sigma, T) to a cheapest augmented
// path in a graph whose vertices are (model, batch size); without its self-loops that graph is acyclic (an
// edge always leads to a strictly smaller model index), so the cheapest path is a cost-to-go recursion:
//   down(i, j) = cheapest expected cost for a sub-hierarchy topped by model i to hand up a batch of j tokens
//              = min( j c_i                                            (model i is the bottom level),
//                     min_{k < i, l <= j} gamma(alpha_{k,i}, l, j) (c_i + down(k, l)) )
//   L*        = min( c_K,  min_{i < K, j} (1 - a) / (1 - a^(j+1)) (c_K + down(i, j)) ),  a = alpha_{i,K}.
int hsd_search_hierarchy(const double *costs, const double *alpha, int n_models, int T_max, int32_t *out_sigma,
                         int32_t *out_n_levels, int32_t *out_T, double *out_latency) {
  if (!costs || !out_sigma || !out_n_levels || n_models < 1 || n_models > 64 || T_max < 1 || T_max > 64)
    return HSD_E_INVALID_ARG;
  const int K = n_models - 1;
  if (K > 0 && (!alpha || !out_T)) return HSD_E_INVALID_ARG;
  for (int i = 0; i < n_models; ++i) {
    if (!(costs[i] >= 0.0)) return HSD_E_INVALID_ARG;
    for (int j = i + 1; j < n_models; ++j)
      if (!(alpha[(size_t)i * n_models + j] >= 0.0 && alpha[(size_t)i * n_models + j] <= 1.0)) return HSD_E_INVALID_ARG;
  }
  struct Node { double cost; int prev_model, prev_T; };     // prev_model < 0: bottom level
  std::vector<Node> down((size_t)(K > 0 ? K : 1) * (T_max + 1));
  auto at = [&](int i, int j) -> Node & { return down[(size_t)i * (T_max + 1) + j]; };
  for (int i = 0; i < K; ++i)
    for (int j = 1; j <= T_max; ++j) {
      Node best = {j * costs[i], -1, 0};
      for (int k = 0; k < i; ++k) {
        const double a = alpha[(size_t)k * n_models + i];
        for (int l = 1; l <= j; ++l) {
          const double c = gamma_rounds(a, l, j) * (costs[i] + at(k, l).cost);
          if (c < best.cost) best = {c, k, l};
        }
      }
      at(i, j) = best;
    }
  double best_l = costs[K];
  int top_model = -1, top_T = 0;
  for (int i = 0; i < K; ++i)
    for (int j = 1; j <= T_max; ++j) {
      const double c = top_multiplier(alpha[(size_t)i * n_models + K], j) * (costs[K] + at(i, j).cost);
      if (c < best_l) { best_l = c; top_model = i; top_T = j; }
    }
  // walk the chain down from the target, then reverse it
  std::vector<int32_t> sig, Ts;
  sig.push_back(K);
  for (int i = top_model, j = top_T; i >= 0;) {
    sig.push_back(i);
    Ts.push_back(j);
    const Node &n = at(i, j);
    i = n.prev_model;
    j = n.prev_T;
  }
  const int n_lev = (int)sig.size();
  for (int k = 0; k < n_lev; ++k) out_sigma[k] = sig[n_lev - 1 - k];
  for (int k = 0; k + 1 < n_lev; ++k) out_T[k] = Ts[n_lev - 2 - k];
  *out_n_levels = n_lev;
  if (out_latency) *out_latency = best_l;
  return HSD_OK;
}

}  // extern "C"

// Host-side cache-pool planner (no CUDA): the paper's Section 3.4 "Compression-Aware
// Cache Management" with Algorithms 2 (probabilistic modelling of cache hits),
// 3 (makespan estimation) and 4 (hierarchical cache pool planning) of its appendix,
// and the modified iterative proportional fitting that turns rank-based inclusion
// probabilities into selection probabilities (appendix on the maximum-entropy
// property).  Pools: 0 = F full tensors, 1 = C compressed, 2 = S SM-chunks, 3 = E E-chunks.
#include <cmath>
#include <cstdint>
#include <vector>

#include "zipmoe.h"

namespace {

// Algorithm 2 on q[lo, hi): phi[h] = P(exactly h of these ranks are selected)
std::vector<double> hit_distribution(const double *q, uint32_t lo, uint32_t hi) {
  const uint32_t m = hi - lo;
  std::vector<double> phi(m + 1, 0.0);
  phi[0] = 1.0;
  for (uint32_t r = 0; r < m; ++r) {
    const double p = q[lo + r];
    for (uint32_t h = r + 1; h >= 1; --h) phi[h] = phi[h] * (1.0 - p) + phi[h - 1] * p;
    phi[0] *= 1.0 - p;
  }
  return phi;
}

// elementary symmetric polynomials R(0..k) of the weights w, leaving out index `skip` (or none if skip >= n)
std::vector<double> symmetric(const std::vector<double> &w, uint32_t k, uint32_t skip) {
  std::vector<double> r(k + 1, 0.0);
  r[0] = 1.0;
  for (uint32_t i = 0; i < w.size(); ++i) {
    if (i == skip) continue;
    for (uint32_t j = k; j >= 1; --j) r[j] += r[j - 1] * w[i];
  }
  return r;
}

bool costs_ok(const zipmoe_plan_costs *c) {
  return c && c->L >= 1 && c->K >= 1 && c->n_tensors >= 1 && c->c >= 0 && c->v >= 0 && c->u >= 0;
}

double makespan(uint32_t k, const uint32_t h[4], const zipmoe_plan_costs &c) {
  const double n = c.n_tensors, K = c.K;
  const double n_sm = n * (double)(k - h[0] - h[1] - h[2]);
  const double n_e = n * K * (double)(k - h[0] - h[1] - h[3]);
  const double n_d = n * K * (double)(k - h[0]);
  const double t_io = n_sm * c.u + n_e * c.v;
  const double t_dec = (n_e * c.v + n_d * c.c) / (double)c.L;
  return t_io > t_dec ? t_io : t_dec;
}

zipmoe_status expected_makespan(const double *q, uint32_t n, uint32_t k, const uint32_t cap[4],
                                const zipmoe_plan_costs &costs, double *expected) {
  uint32_t at = 0;
  std::vector<double> phi[4];
  for (int p = 0; p < 4; ++p) {
    if ((uint64_t)at + cap[p] > n) return ZIPMOE_ERR_INVALID_ARG;
    phi[p] = hit_distribution(q, at, at + cap[p]);
    at += cap[p];
  }
  const std::vector<double> miss = hit_distribution(q, at, n), all = hit_distribution(q, 0, n);
  if (!(all[k] > 0.0)) return ZIPMOE_ERR_INVALID_ARG;   // k experts can not be selected at all
  double cost = 0.0;
  uint32_t h[4];
  for (h[0] = 0; h[0] <= cap[0] && h[0] <= k; ++h[0])
    for (h[1] = 0; h[1] <= cap[1] && h[0] + h[1] <= k; ++h[1])
      for (h[2] = 0; h[2] <= cap[2] && h[0] + h[1] + h[2] <= k; ++h[2])
        for (h[3] = 0; h[3] <= cap[3] && h[0] + h[1] + h[2] + h[3] <= k; ++h[3]) {
          const uint32_t rem = k - h[0] - h[1] - h[2] - h[3];
          if (rem >= miss.size()) continue;   // more misses than there are ranks outside the pools
          const double pr = miss[rem] / all[k] * phi[0][h[0]] * phi[1][h[1]] * phi[2][h[2]] * phi[3][h[3]];
          cost += pr * makespan(k, h, costs);
        }
  *expected = cost;
  return ZIPMOE_OK;
}

zipmoe_status selection_probs(const double *f, uint32_t n, uint32_t k, uint32_t max_iters, double tol, double *q,
                              uint32_t *iters_done) {
  if (!f || !q || n < 2 || n > 512 || k < 1 || k >= n) return ZIPMOE_ERR_INVALID_ARG;
  double sum = 0.0;
  for (uint32_t i = 0; i < n; ++i) {
    if (!(f[i] > 0.0 && f[i] < 1.0)) return ZIPMOE_ERR_INVALID_ARG;
    sum += f[i];
  }
  if (std::fabs(sum - (double)k) > 1e-6) return ZIPMOE_ERR_INVALID_ARG;
  std::vector<double> w(f, f + n), ft(n);
  uint32_t it = 0;
  for (;; ++it) {
    const double denom = symmetric(w, k, n)[k];
    double worst = 0.0;
    for (uint32_t i = 0; i < n; ++i) {
      ft[i] = w[i] * symmetric(w, k - 1, i)[k - 1] / denom;
      worst = std::fmax(worst, std::fabs(ft[i] - f[i]));
    }
    if (worst <= tol || it >= max_iters) break;
    for (uint32_t i = 0; i < n; ++i) w[i] *= f[i] / ft[i];
  }
  for (uint32_t i = 0; i < n; ++i) q[i] = w[i] / (1.0 + w[i]);
  if (iters_done) *iters_done = it;
  return ZIPMOE_OK;
}

}  // namespace

extern "C" {

zipmoe_status zipmoe_plan_hit_distribution(const double *q, uint32_t n, double *phi) {
  if (!phi || (!q && n)) return ZIPMOE_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < n; ++i)
    if (!(q[i] >= 0.0 && q[i] <= 1.0)) return ZIPMOE_ERR_INVALID_ARG;
  const std::vector<double> r = hit_distribution(q, 0, n);
  for (uint32_t h = 0; h <= n; ++h) phi[h] = r[h];
  return ZIPMOE_OK;
}

zipmoe_status zipmoe_plan_selection_probs(const double *f, uint32_t n, uint32_t k, uint32_t max_iters, double tol,
                                          double *q, uint32_t *iters_done) {
  return selection_probs(f, n, k, max_iters, tol, q, iters_done);
}

zipmoe_status zipmoe_plan_makespan(uint32_t k, const uint32_t hits[4], const zipmoe_plan_costs *costs, double *out) {
  if (!hits || !out || !costs_ok(costs)) return ZIPMOE_ERR_INVALID_ARG;
  if ((uint64_t)hits[0] + hits[1] + hits[2] + hits[3] > k) return ZIPMOE_ERR_INVALID_ARG;
  *out = makespan(k, hits, *costs);
  return ZIPMOE_OK;
}

zipmoe_status zipmoe_plan_expected_makespan(const double *q, uint32_t n, uint32_t k, const uint32_t capacity[4],
                                            const zipmoe_plan_costs *costs, double *expected) {
  if (!q || !capacity || !expected || !costs_ok(costs) || k < 1 || k > n) return ZIPMOE_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < n; ++i)
    if (!(q[i] >= 0.0 && q[i] <= 1.0)) return ZIPMOE_ERR_INVALID_ARG;
  return expected_makespan(q, n, k, capacity, *costs, expected);
}

zipmoe_status zipmoe_plan_cache_pools(const double *f, uint32_t n, uint32_t k, uint32_t pool_mask, double budget,
                                      const double expert_size[4], const zipmoe_plan_costs *costs, double step,
                                      double ratios[4], uint32_t capacity[4], double *expected) {
  if (!f || !expert_size || !ratios || !capacity || !expected || !costs_ok(costs)) return ZIPMOE_ERR_INVALID_ARG;
  if (!(pool_mask & 15u) || !(budget >= 0.0) || !(step > 0.0 && step <= 1.0)) return ZIPMOE_ERR_INVALID_ARG;
  const uint32_t G = (uint32_t)std::llround(1.0 / step);
  if (G < 1 || G > 100 || std::fabs(G * step - 1.0) > 1e-9) return ZIPMOE_ERR_INVALID_ARG;
  for (int p = 0; p < 4; ++p)
    if ((pool_mask >> p & 1u) && !(expert_size[p] > 0.0)) return ZIPMOE_ERR_INVALID_ARG;
  std::vector<double> q(n);
  zipmoe_status rc = selection_probs(f, n, k, 1000, 1e-12, q.data(), nullptr);
  if (rc != ZIPMOE_OK) return rc;

  double best = INFINITY;
  uint32_t g[4];
  // every split of G grid steps over the pools in use; pools not in use stay at 0
  for (g[0] = 0; g[0] <= ((pool_mask & 1u) ? G : 0); ++g[0])
    for (g[1] = 0; g[1] <= ((pool_mask & 2u) ? G - g[0] : 0); ++g[1])
      for (g[2] = 0; g[2] <= ((pool_mask & 4u) ? G - g[0] - g[1] : 0); ++g[2]) {
        const uint32_t left = G - g[0] - g[1] - g[2];
        if (!(pool_mask & 8u) && left != 0) continue;   // the ratios must sum to one
        g[3] = (pool_mask & 8u) ? left : 0;
        uint32_t cap[4], used = 0;
        for (int p = 0; p < 4; ++p) {
          double want = g[p] ? std::floor((double)g[p] / G * budget / expert_size[p] + 1e-9) : 0.0;
          uint32_t c = want > (double)(n - used) ? n - used : (uint32_t)want;
          cap[p] = c;
          used += c;
        }
        double cost = 0.0;
        rc = expected_makespan(q.data(), n, k, cap, *costs, &cost);
        if (rc != ZIPMOE_OK) return rc;
        if (cost < best) {
          best = cost;
          for (int p = 0; p < 4; ++p) {
            ratios[p] = (double)g[p] / G;
            capacity[p] = cap[p];
          }
        }
      }
  if (!(best < INFINITY)) return ZIPMOE_ERR_INVALID_ARG;
  *expected = best;
  return ZIPMOE_OK;
}

}  // extern "C"

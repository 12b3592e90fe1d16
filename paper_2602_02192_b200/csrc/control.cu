// Host-side closed forms of the paper's provisioning and staleness rules (no GPU work).
//
// A rollout worker's throughput mu_i (rollouts per second) is what echo_rollout delivers divided by
// the tokens per rollout; these functions turn measured throughputs into the quantities of
// Section 3: the capacity a publication period needs, the conservative staleness bound, the greedy
// cost-ranked activation, and the replay buffer's admission test of Section 4.2.

#include <algorithm>
#include <cmath>
#include <numeric>
#include <vector>

#include "../../include/echo.h"

extern "C" {

int echo_mu_min(double kappa, double R, double T_train, double T_bcast, double *out) {
  if (!out || !(kappa > 0.0) || !(R > 0.0) || !(T_train > 0.0) || !(T_bcast >= 0.0)) return ECHO_ERR_INVALID;
  const double slack = kappa * T_train - T_bcast;          // time left for generation in one period
  if (!(slack > 0.0)) return ECHO_ERR_UNSUPPORTED;         // the overlap condition cannot be met at this kappa
  *out = kappa * R / slack;
  return ECHO_OK;
}

int echo_staleness_bound(int32_t kappa, double T_bcast, double R, double mu_pool, double T_train, int32_t *out) {
  if (!out || kappa < 1 || !(T_bcast >= 0.0) || !(R > 0.0) || !(mu_pool > 0.0) || !(T_train > 0.0))
    return ECHO_ERR_INVALID;
  const double steps = std::ceil((T_bcast + R / mu_pool) / T_train);
  if (!(steps < 2147483647.0 - kappa)) return ECHO_ERR_INVALID;
  *out = kappa + static_cast<int32_t>(steps) - 1;
  return ECHO_OK;
}

int echo_greedy_provision(const double *mu, const double *cost, int32_t n, double mu_target, uint8_t *active,
                          int32_t *n_active, double *total_cost) {
  if (!mu || !cost || !active || n < 0 || !(mu_target >= 0.0)) return ECHO_ERR_INVALID;
  for (int32_t i = 0; i < n; ++i)
    if (!(mu[i] > 0.0) || !(cost[i] >= 0.0)) return ECHO_ERR_INVALID;
  std::vector<int32_t> order(n);
  std::iota(order.begin(), order.end(), 0);
  // increasing unit throughput cost rho_i = c_i / mu_i; equal rho: lower index first
  std::stable_sort(order.begin(), order.end(),
                   [&](int32_t a, int32_t b) { return cost[a] / mu[a] < cost[b] / mu[b]; });
  std::fill(active, active + n, static_cast<uint8_t>(0));
  double cap = 0.0, c = 0.0;
  int32_t k = 0;
  while (cap < mu_target && k < n) {
    active[order[k]] = 1;
    cap += mu[order[k]];
    c += cost[order[k]];
    ++k;
  }
  if (n_active) *n_active = k;
  if (total_cost) *total_cost = c;
  return cap >= mu_target ? ECHO_OK : ECHO_ERR_UNSUPPORTED;   // the whole pool is too slow
}

int echo_admissible(int64_t v, int64_t v_t, int64_t S) { return S >= 0 && v <= v_t && v >= v_t - S ? 1 : 0; }

}  // extern "C"

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

// Appendix C.3 ("Worker scoring").  The Speed term is clamped to [0, 100]: the paper says that it
// saturates at 100 at the per-worker cap; the lower clamp keeps a very slow peer from scoring below
// a peer that has never succeeded.
int echo_peer_score(double avg_speed, double success_rate, int32_t succ_count, int32_t consecutive_failures,
                    double elapsed_s, double *out) {
  if (!out || !(avg_speed >= 0.0) || !(success_rate >= 0.0) || success_rate > 1.0 || succ_count < 0 ||
      consecutive_failures < 0 || !(elapsed_s >= 0.0))
    return ECHO_ERR_INVALID;
  double speed = avg_speed > 0.0 ? 100.0 * (std::log10(avg_speed) - 3.0) / 5.0 : 0.0;
  speed = std::min(100.0, std::max(0.0, speed));
  const double success = 100.0 * success_rate;
  const double stability = consecutive_failures > 3 ? 0.0 : 100.0 * std::min(succ_count / 10.0, 1.0);
  const double decay = 1.0 - std::min(elapsed_s / 600.0, 0.3);
  *out = decay * (0.5 * speed + 0.35 * success + 0.15 * stability);
  return ECHO_OK;
}

// Appendix C.3 ("Chain assembly") with N_ch = floor(B0 / Bw) of Section 4.3, at least one chain and
// at most one per worker.
int echo_chain_assemble(const double *score, int32_t n, double B0, double Bw, int32_t *chain_of, int32_t *hop_of,
                        int32_t *n_chains) {
  if (!score || !chain_of || !hop_of || !n_chains || n < 0 || !(B0 > 0.0) || !(Bw > 0.0)) return ECHO_ERR_INVALID;
  for (int32_t i = 0; i < n; ++i)
    if (!(score[i] == score[i])) return ECHO_ERR_INVALID;           // NaN
  double nch = std::floor(B0 / Bw);
  if (nch < 1.0) nch = 1.0;
  const int32_t N = n == 0 ? 0 : static_cast<int32_t>(std::min<double>(nch, n));
  std::vector<int32_t> order(n);
  std::iota(order.begin(), order.end(), 0);
  // decreasing score; equal scores: lower index first
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return score[a] > score[b]; });
  for (int32_t r = 0; r < n; ++r) {
    chain_of[order[r]] = r % N;          // ranks 0..N-1 seed the chains, the rest go to the tails round-robin
    hop_of[order[r]] = r / N;
  }
  *n_chains = N;
  return ECHO_OK;
}

// Section 4.3: chunked store-and-forward at rate Bw with fan-out 1, as a timeline.  The source holds
// the whole snapshot at time 0; link h carries the chunks in order from the node at hop h - 1 (the
// source for h = 0) to the node at hop h, starts a chunk when it has fully arrived upstream and the
// link has finished the chunk before it, takes size / Bw for it, and the chunk is usable downstream
// hop_latency_s later.  The result is the time at which the node at `hop` holds the last chunk.
// With equal chunks and no latency this is (n_chunks + hop) chunk times: one pipeline fill, then line rate.
int echo_chain_arrival_time(double bytes, double chunk_bytes, double Bw_bytes_per_s, int32_t hop,
                            double hop_latency_s, double *out) {
  if (!out || !(bytes > 0.0) || !(chunk_bytes > 0.0) || !(Bw_bytes_per_s > 0.0) || hop < 0 || !(hop_latency_s >= 0.0))
    return ECHO_ERR_INVALID;
  const double nc = std::ceil(bytes / chunk_bytes);
  if (!(nc * (hop + 1.0) <= 1e9)) return ECHO_ERR_UNSUPPORTED;
  const long n_chunks = static_cast<long>(nc);
  std::vector<double> link_free(hop + 1, 0.0);      // when link h has finished its previous chunk
  double arrived = 0.0;
  for (long k = 0; k < n_chunks; ++k) {
    const double size = k + 1 < n_chunks ? chunk_bytes : bytes - (n_chunks - 1) * chunk_bytes;
    arrived = 0.0;                                  // at the source
    for (int32_t h = 0; h <= hop; ++h) {
      const double start = std::max(arrived, link_free[h]);
      link_free[h] = start + size / Bw_bytes_per_s;
      arrived = link_free[h] + hop_latency_s;
    }
  }
  *out = arrived;
  return ECHO_OK;
}

}  // extern "C"

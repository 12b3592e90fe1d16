"""Provisioning and staleness closed forms (oracle side), plain Python.

Section 3.1: overlap condition kappa T_train >= T_bcast + kappa R / sum(mu) and its
rearrangement mu_min(kappa) = kappa R / (kappa T_train - T_bcast); the conservative
staleness bound Delta_max <= kappa + ceil((T_bcast + R / mu_pool) / T_train) - 1.
Section 3.2: greedy activation of the cheapest prefix by unit throughput cost
rho_i = c_i / mu_i.  Section 4.2: replay admission v >= v_t - S.

Appendix C.3: peer score and chain assembly; Section 4.3: store-and-forward timeline.

Pins: mu_min makes the overlap condition an equality; kappa = 2 with
T_bcast < 2 T_train under the overlap condition gives a bound of at most 3 and
kappa = S - 1 a bound of at most S (Appendix on staleness); the greedy set is a
prefix of the rho ranking, feasible, and minimal as a prefix; on small pools it is
compared with exhaustive search (never cheaper than the optimum, equal to it for
equal-throughput workers).
"""
from __future__ import annotations

import math
from fractions import Fraction


def mu_min(kappa, R, T_train, T_bcast):
    slack = Fraction(kappa) * Fraction(T_train) - Fraction(T_bcast)
    if slack <= 0:
        raise ValueError("kappa * T_train must exceed T_bcast")
    return float(Fraction(kappa) * Fraction(R) / slack)


def staleness_bound(kappa: int, T_bcast, R, mu_pool, T_train) -> int:
    x = (Fraction(T_bcast) + Fraction(R) / Fraction(mu_pool)) / Fraction(T_train)
    return int(kappa) + math.ceil(x) - 1


def greedy_provision(mu, cost, mu_target):
    """Returns (sorted list of active indices, total cost, reached)."""
    order = sorted(range(len(mu)), key=lambda i: (Fraction(cost[i]) / Fraction(mu[i]), i))
    active, cap, c = [], Fraction(0), Fraction(0)
    for i in order:
        if cap >= Fraction(mu_target):
            break
        active.append(i)
        cap += Fraction(mu[i])
        c += Fraction(cost[i])
    return sorted(active), float(c), cap >= Fraction(mu_target)


def admissible(v: int, v_t: int, S: int) -> bool:
    return v_t - S <= v <= v_t


def peer_score(avg_speed, success_rate, succ_count, consecutive_failures, elapsed_s) -> float:
    """Appendix C.3, "Worker scoring", term by term.  avg_speed in bits per second.  Speed is clamped
    to [0, 100] (the appendix: it saturates at 100 at the per-worker cap; below 1 kbit/s: 0)."""
    speed = 100.0 * (math.log10(avg_speed) - 3.0) / 5.0 if avg_speed > 0 else 0.0
    speed = min(100.0, max(0.0, speed))
    success = 100.0 * success_rate
    stability = 0.0 if consecutive_failures > 3 else 100.0 * min(succ_count / 10.0, 1.0)
    decay = 1.0 - min(elapsed_s / 600.0, 0.3)
    return decay * (0.5 * speed + 0.35 * success + 0.15 * stability)


def chain_assemble(scores, B0, Bw):
    """Appendix C.3, "Chain assembly".  Returns the chains as lists of worker indices, seed first:
    N_ch = floor(B0 / Bw) chains (at least one, at most one per worker); the best N_ch workers seed
    them, the rest go to the tails in rank order, round-robin."""
    n = len(scores)
    if n == 0:
        return []
    n_ch = max(1, min(n, int(Fraction(B0) / Fraction(Bw))))
    ranked = sorted(range(n), key=lambda i: (-scores[i], i))
    chains = [[] for _ in range(n_ch)]
    for r, w in enumerate(ranked):
        chains[r % n_ch].append(w)
    return chains


def chain_arrival_time(n_bytes, chunk_bytes, Bw, hop, hop_latency=0.0) -> float:
    """Section 4.3, store-and-forward streaming along a chain, simulated chunk by chunk and link by
    link with exact rationals: when does the worker at `hop` (0 = seed) hold the last chunk."""
    n_bytes, chunk_bytes, Bw, lat = Fraction(n_bytes), Fraction(chunk_bytes), Fraction(Bw), Fraction(hop_latency)
    n_chunks = -(-n_bytes // chunk_bytes)
    sizes = [chunk_bytes] * (n_chunks - 1) + [n_bytes - (n_chunks - 1) * chunk_bytes]
    have = [Fraction(0)] * n_chunks               # when each chunk is complete at the current node (source: 0)
    for _link in range(hop + 1):
        free = Fraction(0)
        nxt = []
        for k, size in enumerate(sizes):
            start = max(have[k], free)
            free = start + size / Bw
            nxt.append(free + lat)
        have = nxt
    return float(have[-1])

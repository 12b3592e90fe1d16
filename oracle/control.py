"""Provisioning and staleness closed forms (oracle side), plain Python.

Section 3.1: overlap condition kappa T_train >= T_bcast + kappa R / sum(mu) and its
rearrangement mu_min(kappa) = kappa R / (kappa T_train - T_bcast); the conservative
staleness bound Delta_max <= kappa + ceil((T_bcast + R / mu_pool) / T_train) - 1.
Section 3.2: greedy activation of the cheapest prefix by unit throughput cost
rho_i = c_i / mu_i.  Section 4.2: replay admission v >= v_t - S.

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

"""Host-side closed forms of Sections 3 and 4.2: oracle pins and the library's C functions (no GPU)."""
import ctypes as C
import itertools
import math

import numpy as np
import pytest

from oracle import control


@pytest.fixture(scope="module")
def lib():
    from paper_2602_02192_b200 import binding
    return binding.lib


def test_mu_min_is_the_overlap_condition_at_equality():
    for kappa, R, Tt, Tb in [(2, 512, 1500.0, 900.0), (1, 64, 10.0, 3.5), (5, 1000, 1600.0, 0.0)]:
        mu = control.mu_min(kappa, R, Tt, Tb)
        assert math.isclose(kappa * Tt, Tb + kappa * R / mu, rel_tol=1e-12)
        assert control.mu_min(kappa, R, Tt, Tb / 2 if Tb else 0.0) <= mu        # less dissemination time, less capacity
    with pytest.raises(ValueError):
        control.mu_min(2, 512, 100.0, 200.0)


def test_staleness_bound_cases_of_the_appendix():
    # kappa = 2, T_bcast < 2 T_train, capacity from the overlap condition: ceiling term <= 2, bound <= 3
    rng = np.random.default_rng(0)
    for _ in range(200):
        Tt = float(rng.uniform(10, 2000))
        Tb = float(rng.uniform(0, 0.999 * Tt))                # T_bcast / T_train < 1
        R = int(rng.integers(1, 4096))
        for S in (2, 3, 5):
            kappa = S - 1
            mu = control.mu_min(kappa, R, Tt, Tb) * float(rng.uniform(1.0, 3.0))
            b = control.staleness_bound(kappa, Tb, R, mu, Tt)
            assert kappa <= b <= S
    assert control.staleness_bound(2, 0.5, 10, 10.0, 1.0) == 2 + 2 - 1      # (0.5 + 1) / 1 -> ceil 2
    assert control.staleness_bound(3, 0.0, 10, 10.0, 1.0) == 3              # exactly one step: ceil 1


def test_greedy_provision_properties_and_exhaustive_search():
    rng = np.random.default_rng(1)
    for _ in range(100):
        n = int(rng.integers(1, 9))
        mu = [float(x) for x in rng.integers(1, 20, size=n)]
        cost = [float(x) for x in rng.integers(1, 30, size=n)]
        target = float(rng.uniform(0.1, 1.1) * sum(mu))
        act, c, ok = control.greedy_provision(mu, cost, target)
        rank = sorted(range(n), key=lambda i: (cost[i] / mu[i], i))
        assert act == sorted(rank[: len(act)])                              # a prefix of the rho ranking
        if not ok:
            assert target > sum(mu) and len(act) == n
            continue
        cap = sum(mu[i] for i in act)
        assert cap >= target and cap - mu[rank[len(act) - 1]] < target      # feasible, minimal as a prefix
        best = min(sum(cost[i] for i in sub) for k in range(n + 1) for sub in itertools.combinations(range(n), k)
                   if sum(mu[i] for i in sub) >= target)
        assert c >= best - 1e-9                                             # greedy, not optimal in general
    # equal throughputs: the cheapest prefix IS the optimum
    mu, cost = [4.0] * 6, [9.0, 2.0, 7.0, 3.0, 8.0, 1.0]
    act, c, ok = control.greedy_provision(mu, cost, 10.0)
    assert ok and act == [1, 3, 5] and c == 6.0


def test_admission_window():
    assert control.admissible(7, 10, 3) and control.admissible(10, 10, 3)
    assert not control.admissible(6, 10, 3) and not control.admissible(11, 10, 3)


def test_library_matches_oracle(lib):
    rng = np.random.default_rng(2)
    out = C.c_double()
    for _ in range(50):
        kappa = int(rng.integers(1, 6)); R = int(rng.integers(1, 2000))
        Tt = float(rng.uniform(1, 2000)); Tb = float(rng.uniform(0, kappa * Tt * 0.99))
        assert lib.echo_mu_min(kappa, R, Tt, Tb, C.byref(out)) == 0
        assert math.isclose(out.value, control.mu_min(kappa, R, Tt, Tb), rel_tol=1e-12)
        b = C.c_int32()
        mu = float(rng.uniform(0.01, 50))
        assert lib.echo_staleness_bound(kappa, Tb, R, mu, Tt, C.byref(b)) == 0
        assert b.value == control.staleness_bound(kappa, Tb, R, mu, Tt)
    assert lib.echo_mu_min(2.0, 512.0, 100.0, 200.0, C.byref(out)) != 0
    assert lib.echo_mu_min(0.0, 512.0, 100.0, 20.0, C.byref(out)) != 0
    for _ in range(50):
        n = int(rng.integers(1, 12))
        mu = rng.integers(1, 20, size=n).astype(np.float64)
        cost = rng.integers(0, 30, size=n).astype(np.float64)
        target = float(rng.uniform(0.1, 1.2) * mu.sum())
        active = np.zeros(n, dtype=np.uint8)
        k, c = C.c_int32(), C.c_double()
        rc = lib.echo_greedy_provision(mu.ctypes.data_as(C.POINTER(C.c_double)),
                                       cost.ctypes.data_as(C.POINTER(C.c_double)), n, target,
                                       active.ctypes.data_as(C.POINTER(C.c_uint8)), C.byref(k), C.byref(c))
        act, want_c, ok = control.greedy_provision(list(mu), list(cost), target)
        assert (rc == 0) == ok and sorted(np.flatnonzero(active)) == act and k.value == len(act)
        assert math.isclose(c.value, want_c, rel_tol=1e-12, abs_tol=1e-12)
    for v, vt, S in [(7, 10, 3), (6, 10, 3), (10, 10, 0), (11, 10, 3), (5, 5, -1)]:
        assert lib.echo_admissible(v, vt, S) == int(S >= 0 and control.admissible(v, vt, S))

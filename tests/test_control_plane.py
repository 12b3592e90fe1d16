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


# ---- Appendix C.3: peer score, chain assembly; Section 4.3: store-and-forward timeline ---------------

def test_peer_score_facts_of_the_appendix():
    # Speed saturates at 100 when the forwarding rate reaches 100 Mbit/s (log10 = 8)
    best = control.peer_score(1e8, 1.0, 10, 0, 0.0)
    assert math.isclose(best, 100.0, rel_tol=1e-12)
    assert control.peer_score(1e9, 1.0, 10, 0, 0.0) == best                    # no credit beyond the cap
    # weights 0.5 / 0.35 / 0.15, each term alone
    assert math.isclose(control.peer_score(1e8, 0.0, 0, 0, 0.0), 50.0)
    assert math.isclose(control.peer_score(1e3, 1.0, 0, 0, 0.0), 35.0)          # log10 = 3: Speed 0
    assert math.isclose(control.peer_score(1e3, 0.0, 10, 0, 0.0), 15.0)
    assert math.isclose(control.peer_score(1e3, 0.0, 5, 3, 0.0), 7.5)           # 5 of 10 successes, 3 failures still count
    assert control.peer_score(1e3, 0.0, 10, 4, 0.0) == 0.0                      # more than 3 consecutive failures
    # Speed is linear in log10 between 1 kbit/s and the cap: 10^5.5 is half way
    assert math.isclose(control.peer_score(10 ** 5.5, 0.0, 0, 0, 0.0), 25.0, rel_tol=1e-12)
    # Decay: 1 at once, 0.85 after 90 s, floor 0.7 from 180 s on
    assert math.isclose(control.peer_score(1e8, 1.0, 10, 0, 90.0), 85.0)
    assert math.isclose(control.peer_score(1e8, 1.0, 10, 0, 180.0), 70.0)
    assert control.peer_score(1e8, 1.0, 10, 0, 1e6) == control.peer_score(1e8, 1.0, 10, 0, 180.0)


def test_chain_assembly_rules():
    scores = [10.0, 90.0, 50.0, 70.0, 30.0, 70.0, 20.0]
    chains = control.chain_assemble(scores, 300.0, 100.0)                        # floor(300 / 100) = 3 chains
    assert [c[0] for c in chains] == [1, 3, 5]                                  # the three best seed them (tie: lower index)
    # ranking: 1 (90), 3 and 5 (70), 2 (50), 4 (30), 6 (20), 0 (10); ranks 3.. go to chains 0, 1, 2, 0, ...
    assert chains == [[1, 2, 0], [3, 4], [5, 6]]
    flat = sorted(w for c in chains for w in c)
    assert flat == list(range(len(scores)))                                     # every worker in exactly one chain
    assert len(control.chain_assemble(scores, 50.0, 100.0)) == 1                # an uplink below one worker's rate: one chain
    assert len(control.chain_assemble(scores, 1e9, 100.0)) == len(scores)       # never more chains than workers (a star)
    assert control.chain_assemble([], 300.0, 100.0) == []


def test_store_and_forward_timeline_closed_forms():
    Bw = 100.0
    # one chunk: pure store and forward, the whole snapshot crosses hop + 1 links one after the other
    assert math.isclose(control.chain_arrival_time(1000, 1000, Bw, 3), 4 * 10.0)
    # equal chunks: (n_chunks + hop) chunk times - a pipeline fill, then line rate
    for n_chunks, hop in [(10, 0), (10, 4), (64, 7), (1, 5)]:
        t = control.chain_arrival_time(100 * n_chunks, 100, Bw, hop)
        assert math.isclose(t, (n_chunks + hop) * 1.0)
    # finer chunks approach the line rate bytes / Bw whatever the hop
    assert control.chain_arrival_time(10000, 1, Bw, 7) < 100.0 * 1.001
    # a shorter last chunk: brute force against the recurrence written out by hand for 2 chunks, 2 links
    # sizes 100 and 50: link 0 ends them at 1.0 and 1.5; link 1 starts them at 1.0 and max(1.5, 2.0), ends at 2.5
    assert math.isclose(control.chain_arrival_time(150, 100, Bw, 1), 2.5)
    # per-hop latency is paid once per link by the last chunk when the links are otherwise idle for it
    assert math.isclose(control.chain_arrival_time(100, 100, Bw, 2, hop_latency=0.25), 3 * (1.0 + 0.25))
    # a deeper hop never holds the snapshot earlier
    ts = [control.chain_arrival_time(12345, 1000, Bw, h, 0.01) for h in range(6)]
    assert all(b > a for a, b in zip(ts, ts[1:]))


def test_library_peer_score_chains_and_timeline_match_the_oracle(lib):
    rng = np.random.default_rng(5)
    out = C.c_double()
    for _ in range(300):
        a = (float(10 ** rng.uniform(1, 10)), float(rng.uniform(0, 1)), int(rng.integers(0, 25)),
             int(rng.integers(0, 7)), float(rng.uniform(0, 1200)))
        assert lib.echo_peer_score(*a, C.byref(out)) == 0
        assert math.isclose(out.value, control.peer_score(*a), rel_tol=1e-12, abs_tol=1e-12)
    assert lib.echo_peer_score(0.0, 0.5, 3, 0, 0.0, C.byref(out)) == 0 and math.isclose(out.value, 0.35 * 50 + 0.15 * 30)
    assert lib.echo_peer_score(1e6, 1.5, 3, 0, 0.0, C.byref(out)) == -1
    for _ in range(100):
        n = int(rng.integers(0, 40))
        scores = np.round(rng.uniform(0, 100, size=n), 0)                        # rounded: ties happen
        B0, Bw = float(rng.uniform(50, 2000)), float(rng.choice([50.0, 100.0, 300.0]))
        chain_of = (C.c_int32 * max(n, 1))()
        hop_of = (C.c_int32 * max(n, 1))()
        n_ch = C.c_int32()
        rc = lib.echo_chain_assemble(scores.ctypes.data_as(C.POINTER(C.c_double)), n, B0, Bw, chain_of, hop_of,
                                     C.byref(n_ch))
        assert rc == 0
        want = control.chain_assemble(list(scores), B0, Bw)
        assert n_ch.value == len(want)
        for c, chain in enumerate(want):
            for h, w in enumerate(chain):
                assert chain_of[w] == c and hop_of[w] == h
    for _ in range(200):
        n_bytes = float(rng.integers(1, 10 ** 7))
        chunk = float(rng.integers(1, 10 ** 6))
        Bw, hop, lat = float(rng.uniform(1e3, 1e6)), int(rng.integers(0, 12)), float(rng.uniform(0, 0.01))
        assert lib.echo_chain_arrival_time(n_bytes, chunk, Bw, hop, lat, C.byref(out)) == 0
        assert math.isclose(out.value, control.chain_arrival_time(n_bytes, chunk, Bw, hop, lat), rel_tol=1e-9)

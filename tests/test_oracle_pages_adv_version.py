"""Pins for the oracle's page plan, group advantage and version state machine."""
import os

import numpy as np
import pytest

from oracle import advantage, pages, version

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- page plan
@pytest.mark.parametrize("lens,G,T,Z", [
    ([32, 32, 32, 32], 4, 32, 16),
    ([20, 33, 16, 1], 3, 9, 16),
    ([5], 2, 1, 16),
    ([17, 31], 2, 40, 8),
])
def test_page_plan_bruteforce(lens, G, T, Z):
    plan = pages.build(lens, G, T, Z)
    P = len(lens)
    seen = {}
    for p in range(P):
        full = (lens[p] // Z) * Z
        for g in range(G):
            s = p * G + g
            for t in range(lens[p] + T - 1):
                pg, off = pages.slot(plan, s, t)
                assert 0 <= pg < plan.n_pages and 0 <= off < Z
                key = (pg, off)
                if t < full:
                    # shared by exactly the samples of this group at the same t
                    assert seen.setdefault(key, (p, t)) == (p, t)
                else:
                    assert key not in seen, "private slot reused"
                    seen[key] = (s, t, "private")
    # prefill writes: full pages coincide with the shared ones, the partial page is its own
    for p in range(P):
        for t in range(lens[p]):
            pg = plan.prefill_table[p, t // Z]
            assert pg >= 0
            if t < (lens[p] // Z) * Z:
                assert pg == plan.table[p * G, t // Z]
            else:
                assert all(pg != plan.table[p * G + g, t // Z] for g in range(G))
    # every physical page is referenced
    used = set(plan.table[plan.table >= 0].tolist()) | set(plan.prefill_table[plan.prefill_table >= 0].tolist())
    assert used == set(range(plan.n_pages))


def test_page_plan_closed_form_counts():
    # 8B-shape workload: 32 prompts x G=8, Lp=512, T=2048, pages of 16 tokens
    plan = pages.build([512] * 32, 8, 2048, 16)
    n_pre, n_dec = 32, (512 + 2047 + 15) // 16 - 32
    assert plan.n_pages == 32 * n_pre + 256 * n_dec
    assert plan.width == 160
    assert plan.table[0, 0] == 0 and plan.table[8, 0] == n_pre
    assert plan.table[3, 31] == 31 and plan.table[3, 32] == 32 * n_pre + 3 * n_dec
    assert np.all(plan.table >= 0)


# ---------------------------------------------------------------- advantage
def _cases():
    out = []
    with open(os.path.join(GOLDEN, "group_advantage_cases.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            a, b = line.split("|")
            out.append(([float(x) for x in a.split()], [float(x) for x in b.split()]))
    return out


def test_advantage_worked_examples():
    cases = _cases()
    assert len(cases) == 4
    for r, want in cases:
        got = advantage.group_advantage([r])[0]
        assert np.allclose(got, want, rtol=0, atol=1e-12)


def test_advantage_invariants():
    rng = np.random.default_rng(3)
    r = rng.random((16, 8))
    a = advantage.group_advantage(r)
    assert np.allclose(a.sum(axis=1), 0, atol=1e-12)
    sigma = r.std(axis=1, ddof=1)
    assert np.allclose(a.std(axis=1, ddof=1), sigma / (sigma + 1e-6), rtol=1e-12)
    # shift invariance, and near scale invariance (eps breaks it slightly, in a known way)
    assert np.allclose(advantage.group_advantage(r + 7.5), a, atol=1e-9)
    a3 = advantage.group_advantage(3 * r)
    assert np.allclose(a3, a * (sigma + 1e-6)[:, None] / (sigma + 1e-6 / 3)[:, None], rtol=1e-12)
    # a biased (n divisor) std would give a different, larger answer
    biased = (r - r.mean(1, keepdims=True)) / (r.std(axis=1, ddof=0, keepdims=True) + 1e-6)
    assert not np.allclose(a, biased, rtol=1e-3)
    # groups are independent of each other
    assert np.allclose(advantage.group_advantage(r[3:4]), a[3:4])


def test_advantage_rejects_single_sample_groups():
    with pytest.raises(ValueError):
        advantage.group_advantage(np.ones((4, 1)))


# ---------------------------------------------------------------- versions
def test_version_overlapping_install_keeps_old_tag():
    w = version.WorkerVersions(2)
    with pytest.raises(version.NoPolicy):
        w.begin_rollout()
    w.offer(0)
    assert w.begin_rollout() == 0          # nothing else to serve: waits for the install
    w.offer(1)
    assert w.begin_rollout() == 0          # install of 1 still running
    assert w.begin_rollout() == 0
    w.install_complete()
    assert w.begin_rollout() == 1          # picked up at the next rollout start
    assert w.begin_rollout() == 1


def test_version_strictly_increasing_and_busy():
    w = version.WorkerVersions(2)
    w.offer(3)
    w.begin_rollout()
    with pytest.raises(version.BadVersion):
        w.offer(3)
    with pytest.raises(version.BadVersion):
        w.offer(2)
    w.offer(4)
    with pytest.raises(version.Busy):
        w.offer(5)                          # a third live version
    w.install_complete()
    assert w.begin_rollout() == 4
    w.offer(5)
    w.install_complete()
    assert w.begin_rollout() == 5


def test_version_single_buffer_blocks():
    w = version.WorkerVersions(1)
    w.offer(0)
    assert w.begin_rollout() == 0
    w.offer(1)
    assert w.begin_rollout() == 1           # single buffer: old weights are gone

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


# ---- GRPO surrogate with truncated importance sampling (Appendix F) ----------------------------

def test_grpo_surrogate_closed_forms():
    from oracle import objective
    T = 5
    lp = np.log(np.array([[0.2, 0.5, 0.1, 0.7, 0.3]]))
    ones = np.ones((1, T))
    # same policy everywhere: rho = w = 1, J = A
    for A in (1.5, -0.7, 0.0):
        assert np.allclose(objective.grpo_surrogate(lp, lp, lp, [A], ones, 0.2, 2.0), [A], atol=1e-15)
    # the four clipping cases, one token: rho = 1.5 / 0.5 against eps = 0.2
    up, down = lp + np.log(1.5), lp + np.log(0.5)
    one = np.zeros((1, T)); one[0, 2] = 1
    J = lambda new, A: float(objective.grpo_surrogate(new, lp, lp, [A], one, 0.2, 2.0)[0])
    assert np.isclose(J(up, 2.0), 1.2 * 2.0)        # A > 0, rho above the clip: capped
    assert np.isclose(J(down, 2.0), 0.5 * 2.0)      # A > 0, rho below: the unclipped (smaller) branch
    assert np.isclose(J(up, -2.0), 1.5 * -2.0)      # A < 0, rho above: the unclipped (more negative) branch
    assert np.isclose(J(down, -2.0), 0.8 * -2.0)    # A < 0, rho below the clip: capped
    # truncated importance ratio: learner / sampler = 3 capped at C = 2; 0.5 passes through
    samp_lo, samp_hi = lp - np.log(3.0), lp + np.log(2.0)
    assert np.allclose(objective.grpo_surrogate(lp, lp, samp_lo, [1.0], ones, 0.2, 2.0), [2.0])
    assert np.allclose(objective.grpo_surrogate(lp, lp, samp_hi, [1.0], ones, 0.2, 2.0), [0.5])
    # the mask selects and normalises: two of five tokens with weights 2 and 0.5 -> mean 1.25
    mixed = lp.copy(); mixed[0, 0] -= np.log(3.0); mixed[0, 1] += np.log(2.0)
    mk = np.array([[1, 1, 0, 0, 0]])
    assert np.allclose(objective.grpo_surrogate(lp, lp, mixed, [1.0], mk, 0.2, 2.0), [1.25])
    assert np.allclose(objective.grpo_surrogate(lp, lp, mixed, [1.0], np.zeros((1, T)), 0.2, 2.0), [0.0])
    with pytest.raises(ValueError):
        objective.grpo_surrogate(lp, lp, lp, [1.0, 2.0], ones, 0.2, 2.0)


def test_grpo_surrogate_against_vector_formula():
    from oracle import objective
    rng = np.random.default_rng(3)
    n, T = 7, 33
    ln, lo, ls = (-rng.exponential(1.0, size=(n, T)) for _ in range(3))
    adv = rng.normal(size=n)
    mask = (rng.random((n, T)) < 0.6).astype(np.float64)
    mask[3] = 0
    got = objective.grpo_surrogate(ln, lo, ls, adv, mask, 0.2, 1.7)
    rho = np.exp(ln - lo)
    w = np.minimum(np.exp(lo - ls), 1.7)
    term = np.minimum(rho * adv[:, None], np.clip(rho, 0.8, 1.2) * adv[:, None])
    den = mask.sum(1)
    want = np.where(den > 0, (mask * w * term).sum(1) / np.maximum(den, 1), 0.0)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-15)


def test_kl_estimate_and_regularised_objective():
    """Appendix F, the KL term of J-bar.  The per-token estimate is 0 for equal policies, positive
    otherwise, and its mean over tokens drawn from pi_theta is the textbook divergence
    sum_v pi_theta(v) log(pi_theta(v) / pi_ref(v)) (written out here over whole small distributions)."""
    from oracle import objective
    rng = np.random.default_rng(11)
    for V in (2, 5, 17):
        p = rng.dirichlet(np.ones(V))
        q = rng.dirichlet(np.ones(V))
        k = objective.kl_token_estimate(np.log(p), np.log(q))
        assert np.all(k > 0) and np.allclose(objective.kl_token_estimate(np.log(p), np.log(p)), 0.0, atol=1e-15)
        exact = sum(p[v] * (np.log(p[v]) - np.log(q[v])) for v in range(V))
        assert np.isclose(float(np.dot(p, k)), exact, rtol=1e-12)
        # the other direction is a different number: an estimator with the operands swapped fails this
        assert not np.isclose(float(np.dot(p, objective.kl_token_estimate(np.log(q), np.log(p)))), exact, rtol=1e-3)
    # one hand-worked value: pi_ref / pi_theta = 2 -> 2 - ln 2 - 1
    assert np.isclose(objective.kl_token_estimate([np.log(0.25)], [np.log(0.5)])[0], 1.0 - np.log(2.0))
    # in the objective: A = 0 leaves -beta * masked mean of k (w = 1); beta = 0 gives the surrogate back
    T = 6
    ln, lo, ls, lr = (-rng.exponential(1.0, size=(3, T)) for _ in range(4))
    mask = np.array([[1, 1, 0, 1, 0, 0], [0] * 6, [1] * 6], dtype=np.float64)
    adv = np.array([0.7, -1.0, 2.0])
    k = objective.kl_token_estimate(ln, lr)
    got = objective.grpo_objective(ln, lo, lo, lr, np.zeros(3), mask, 0.2, 2.0, 0.3)
    assert np.allclose(got, [-0.3 * k[0, [0, 1, 3]].mean(), 0.0, -0.3 * k[2].mean()])
    assert np.allclose(objective.grpo_objective(ln, lo, ls, lr, adv, mask, 0.2, 1.7, 0.0),
                       objective.grpo_surrogate(ln, lo, ls, adv, mask, 0.2, 1.7))
    # the truncated ratio multiplies the regulariser too (it multiplies the whole of J-bar): w = 2 doubles it
    assert np.allclose(objective.grpo_objective(ln, lo, lo - np.log(3.0), lr, np.zeros(3), mask, 0.2, 2.0, 0.3), 2 * got)
    with pytest.raises(ValueError):
        objective.grpo_objective(ln, lo, ls, lr, adv, mask, 0.2, 1.7, -0.1)


def test_turn_mask_hand_written_dialogue():
    """Appendix F, turn-aware masking, on a dialogue written out by hand.  S = the turn-start id.
    turns: system (c = 1), user (2), assistant (3), user (4), assistant (5): the mask selects turns 3 and 5,
    the turn-start tokens of those turns included (c_t counts the token at t itself)."""
    from oracle import objective
    S = 9
    x = np.array([[S, 1, 2, S, 3, S, 4, 5, 6, S, 7, S, 8, 8]])
    want = np.array([[0, 0, 0, 0, 0, 1, 1, 1, 1, 0, 0, 1, 1, 1]], dtype=np.uint8)
    assert np.array_equal(objective.turn_mask(x, S), want)
    # aligned with next-token targets y_t = x_{t+1}: shifted left by one, last column empty
    shifted = objective.turn_mask(x, S, shift_to_targets=True)
    assert np.array_equal(shifted[:, :-1], want[:, 1:]) and shifted[0, -1] == 0
    # no turn-start token, or only the system turn: nothing to learn from
    assert objective.turn_mask(np.array([[1, 2, 3, 4]]), S).sum() == 0
    assert objective.turn_mask(np.array([[S, 2, 3, 4]]), S).sum() == 0
    # the mask depends on the turn index only: other ids are irrelevant
    y = x.copy()
    y[x != S] = 5
    assert np.array_equal(objective.turn_mask(y, S), want)
    # rows are independent
    two = np.concatenate([x, np.array([[1, S, 2, S, 2, S, 2, 2, S, 1, 1, 1, 1, S]])])
    got = objective.turn_mask(two, S)
    assert np.array_equal(got[0], want[0])
    assert np.array_equal(got[1], np.array([0, 0, 0, 0, 0, 1, 1, 1, 0, 0, 0, 0, 0, 1], dtype=np.uint8))

"""Pins for the oracle's Philox generator, uniform/Gumbel map and sampler."""
import math
import os

import numpy as np
import pytest

from oracle import philox, sampler

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bigint_philox(ctr, key):
    """Independent pure-Python evaluation of the published Philox4x32-10 rounds."""
    c = list(ctr)
    k = list(key)
    for r in range(10):
        if r > 0:
            k[0] = (k[0] + 0x9E3779B9) % (1 << 32)
            k[1] = (k[1] + 0xBB67AE85) % (1 << 32)
        prod0 = 0xD2511F53 * c[0]
        prod1 = 0xCD9E8D57 * c[2]
        c = [(prod1 >> 32) ^ c[1] ^ k[0], prod1 % (1 << 32),
             (prod0 >> 32) ^ c[3] ^ k[1], prod0 % (1 << 32)]
    return c


def _kat_rows():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            v = [int(x, 16) for x in line.split()]
            rows.append((v[:4], v[4:6], v[6:]))
    return rows


def test_philox_known_answers():
    rows = _kat_rows()
    assert len(rows) == 3
    for ctr, key, want in rows:
        got = philox.philox4x32_10(*ctr, *key)
        assert [int(g) for g in got] == want
        assert _bigint_philox(ctr, key) == want


def test_philox_vectorised_matches_bigint_on_random_tuples():
    rng = np.random.default_rng(7)
    c = rng.integers(0, 1 << 32, size=(200, 4), dtype=np.uint64)
    k = rng.integers(0, 1 << 32, size=(200, 2), dtype=np.uint64)
    out = philox.philox4x32_10(c[:, 0], c[:, 1], c[:, 2], c[:, 3], k[:, 0], k[:, 1])
    for i in range(200):
        want = _bigint_philox([int(x) for x in c[i]], [int(x) for x in k[i]])
        assert [int(o[i]) for o in out] == want


def test_philox_counter_to_output_is_injective():
    n = 1 << 16
    out = philox.philox4x32_10(np.arange(n), 3, 5, 0, 0x1234, 0x9)
    packed = set(zip(*(o.tolist() for o in out)))
    assert len(packed) == n


def test_noise_words_layout():
    seed, s, j, V = (0xABCDEF12 << 32) | 0x3456789A, 11, 5, 103
    words = philox.noise_words(seed, s, j, V)
    assert words.shape == (V,) and words.dtype == np.uint32
    for v in (0, 1, 2, 3, 4, 57, 102):
        want = _bigint_philox([v >> 2, j, s, 0], [seed & 0xFFFFFFFF, seed >> 32])[v & 3]
        assert int(words[v]) == want
    # depends on (seed, s, j) each
    assert not np.array_equal(words, philox.noise_words(seed + 1, s, j, V))
    assert not np.array_equal(words, philox.noise_words(seed, s + 1, j, V))
    assert not np.array_equal(words, philox.noise_words(seed, s, j + 1, V))


def test_uniform_range_and_exact_values():
    x = np.array([0, 1, 2, (1 << 24) - 1, 1 << 24, (1 << 31), 0xFFFFFF7F, 0xFFFFFFFF], dtype=np.uint32)
    w = philox.uniform_from_word(x)
    assert w.dtype == np.float32
    assert w[0] == np.float32(2.0 ** -33)
    assert w[1] == np.float32(1.5 * 2.0 ** -32)
    assert w[-1] == np.float32(1.0)
    assert np.all(w > 0) and np.all(w <= 1)
    assert np.all(np.diff(w.astype(np.float64)) >= 0)


def test_uniform_moments():
    words = philox.philox4x32_10(np.arange(1 << 18), 0, 0, 0, 99, 0)
    w = philox.uniform_from_word(np.concatenate(words)).astype(np.float64)
    n = w.size
    assert abs(w.mean() - 0.5) < 4 * math.sqrt(1 / 12 / n)
    assert abs(w.var() - 1 / 12) < 1e-3


def test_gumbel_closed_form_points():
    # w = 1 - 1/e  ->  E = 1  ->  g = 0 ;  w = 1 -> -inf
    g = philox.gumbel_from_uniform(np.array([1 - math.exp(-1.0), 1.0]))
    assert abs(g[0]) < 1e-12
    assert g[1] == -np.inf
    # Gumbel mean is the Euler-Mascheroni constant, variance pi^2/6
    words = philox.philox4x32_10(np.arange(1 << 18), 1, 2, 0, 5, 6)
    gg = philox.gumbel_from_uniform(philox.uniform_from_word(np.concatenate(words)))
    gg = gg[np.isfinite(gg)]
    assert abs(gg.mean() - 0.5772156649) < 0.01
    assert abs(gg.var() - math.pi ** 2 / 6) < 0.03


def test_logprobs_normalised_and_nonpositive():
    rng = np.random.default_rng(0)
    z = rng.normal(size=1000) * 3
    for T in (0.5, 1.0, 2.0):
        d = sampler.draw(z, T, seed=1, s=0, j=0)
        assert abs(np.exp(d.logprobs).sum() - 1) < 1e-12
        assert np.all(d.logprobs <= 0)
        assert d.logprob == d.logprobs[d.token]
        # brute-force argmax of the perturbed scores
        pert = z / T + philox.gumbel_noise(1, 0, 0, len(z))
        best = max(range(len(z)), key=lambda v: (pert[v], -v))
        assert d.token == best
        second = sorted(pert)[-2]
        assert abs(d.margin - (pert[best] - second)) < 1e-12


def test_temperature_scales_distribution():
    z = np.array([0.0, math.log(2.0)])
    d1 = sampler.draw(z, 1.0, 0, 0, 0)
    assert np.allclose(np.exp(d1.logprobs), [1 / 3, 2 / 3])
    d2 = sampler.draw(z, 0.5, 0, 0, 0)          # s = 2z -> probabilities 1/5, 4/5
    assert np.allclose(np.exp(d2.logprobs), [0.2, 0.8])


def test_tie_goes_to_lowest_id():
    z = np.array([1.0, 3.0, 3.0, 0.0])
    g = np.zeros(4)
    d = sampler.draw_with_noise(z, 1.0, g)
    assert d.token == 1 and d.runner_up == 2 and d.margin == 0.0


def test_temperature_must_be_positive():
    with pytest.raises(ValueError):
        sampler.draw(np.zeros(4), 0.0, 0, 0, 0)


def test_gumbel_max_frequencies_match_softmax():
    """Over many independent streams the drawn ids follow softmax(z/T)."""
    z = np.array([0.3, -1.2, 2.0, 0.0, 1.1, -0.4, 0.9, -2.5])
    T = 0.8
    p = np.exp(sampler.log_softmax(z / T))
    n = 20000
    counts = np.zeros(len(z))
    # vary sequence id and step; fixed seed
    for s in range(200):
        for j in range(n // 200):
            counts[sampler.draw(z, T, seed=1234, s=s, j=j).token] += 1
    chi2 = float(((counts - n * p) ** 2 / (n * p)).sum())
    assert chi2 < 24.3          # chi-square, 7 dof, p = 1e-3


# ---- nucleus (top-p) sampling ------------------------------------------------------------------

def test_nucleus_worked_example_and_renormalised_logprob():
    """p = (0.5, 0.3, 0.15, 0.05): top_p 0.9 keeps three tokens (0.8 < 0.9 <= 0.95), top_p 0.8 two,
    top_p 0.5 one; the log-probabilities are those of p / mass."""
    p = np.array([0.3, 0.05, 0.5, 0.15])
    z = np.log(p)
    for top_p, keep in [(0.9, [0, 2, 3]), (0.8, [0, 2]), (0.5, [2]), (0.95, [0, 2, 3]), (0.96, [0, 1, 2, 3])]:
        m = sampler.nucleus_mask(sampler.log_softmax(z), top_p)
        assert sorted(np.flatnonzero(m)) == keep, (top_p, np.flatnonzero(m))
        d = sampler.draw(z, 1.0, 7, 0, 0, top_p)
        mass = p[keep].sum()
        assert d.nucleus_size == len(keep) and math.isclose(d.nucleus_mass, mass, rel_tol=1e-12)
        assert d.token in keep and math.isclose(d.logprob, math.log(p[d.token] / mass), rel_tol=1e-12, abs_tol=1e-12)
        assert math.isclose(np.exp(d.logprobs[m]).sum(), 1.0, rel_tol=1e-12) and np.all(np.isneginf(d.logprobs[~m]))


def test_nucleus_limits_ties_and_nesting():
    rng = np.random.default_rng(5)
    z = rng.normal(size=50)
    full = sampler.draw(z, 0.7, 3, 2, 1)
    same = sampler.draw(z, 0.7, 3, 2, 1, top_p=1.0)
    assert full.token == same.token and full.logprob == same.logprob and same.nucleus_size == 50
    # a vanishing top_p keeps only the most probable token, whatever the noise
    for j in range(20):
        d = sampler.draw(z, 0.7, 3, 2, j, top_p=1e-9)
        assert d.token == int(np.argmax(z)) and abs(d.logprob) < 1e-12 and d.nucleus_size == 1
    # equal probabilities at the boundary: the lower id enters first
    zt = np.log(np.array([0.4, 0.2, 0.2, 0.2]))
    assert sorted(np.flatnonzero(sampler.nucleus_mask(sampler.log_softmax(zt), 0.55))) == [0, 1]
    assert sorted(np.flatnonzero(sampler.nucleus_mask(sampler.log_softmax(zt), 0.65))) == [0, 1, 2]
    # nuclei are nested in top_p, and each is the smallest top-k set that reaches the mass
    lp = sampler.log_softmax(z)
    p = np.exp(lp)
    prev = np.zeros(50, dtype=bool)
    for top_p in (0.1, 0.3, 0.5, 0.9, 0.99):
        m = sampler.nucleus_mask(lp, top_p)
        assert np.all(m[prev]) and p[m].sum() >= top_p
        assert p[m].min() >= p[~m].max()                    # a top-k set
        assert p[m].sum() - p[m].min() < top_p              # dropping its least likely member falls short
        prev = m
    with pytest.raises(ValueError):
        sampler.nucleus_mask(lp, 0.0)


def test_nucleus_frequencies_match_renormalised_distribution():
    z = np.array([0.3, -1.2, 2.0, 0.0, 1.1, -0.4, 0.9, -2.5])
    T, top_p = 0.8, 0.9
    lp = sampler.log_softmax(z / T)
    m = sampler.nucleus_mask(lp, top_p)
    q = np.where(m, np.exp(lp), 0.0)
    q /= q.sum()
    n = 20000
    counts = np.zeros(len(z))
    for s in range(200):
        for j in range(n // 200):
            counts[sampler.draw(z, T, seed=99, s=s, j=j, top_p=top_p).token] += 1
    assert np.all(counts[~m] == 0)
    k = int(m.sum())
    chi2 = float(((counts[m] - n * q[m]) ** 2 / (n * q[m])).sum())
    assert k >= 3 and chi2 < {2: 13.8, 3: 16.3, 4: 18.5, 5: 20.5, 6: 22.5, 7: 24.3}[k - 1]    # p = 1e-3

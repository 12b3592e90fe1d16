"""Pins for the oracle's decoder: closed forms, a scalar-loop evaluation of a
hand-sized model, and agreement of the cached / recompute / teacher-forced modes."""
import math

import numpy as np
import pytest

from oracle import decoder, sampler
from paper_2602_02192_b200 import synth


def _dims(shape):
    return decoder.ModelDims(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads,
                             shape.head_dim, shape.d_ff, shape.vocab, shape.rms_eps, shape.rope_theta)


# ---------------------------------------------------------------- closed forms
def test_widen_bf16_exact():
    bits = np.array([0x3F80, 0xBF80, 0x4000, 0x3DCD, 0x0000, 0x7F80], dtype=np.uint16)
    v = decoder.widen_bf16(bits)
    assert v[0] == 1.0 and v[1] == -1.0 and v[2] == 2.0 and v[4] == 0.0 and np.isinf(v[5])
    assert v[3] == 0.10009765625            # 0x3DCD = 1.6015625 * 2^-4


def test_rmsnorm_closed_forms():
    g = np.array([1.0, 2.0, 3.0, 4.0])
    assert np.allclose(decoder.rmsnorm(np.full(4, 5.0), g, 0.0), g)
    assert np.allclose(decoder.rmsnorm(np.full(4, -5.0), g, 0.0), -g)
    x = np.array([3.0, 4.0, 0.0, 0.0])      # mean square 25/4
    assert np.allclose(decoder.rmsnorm(x, np.ones(4), 0.0), x / 2.5)
    # eps sits inside the square root, added to the mean square
    assert np.allclose(decoder.rmsnorm(x, np.ones(4), 2.75), x / 3.0)


def test_rope_properties():
    rng = np.random.default_rng(0)
    hd, theta = 8, 1e4
    q = rng.normal(size=(1, hd))
    k = rng.normal(size=(1, hd))
    assert np.allclose(decoder.rope(q, 0, theta), q)                 # pos 0 is the identity
    for pos in (1, 7, 100):
        r = decoder.rope(q, pos, theta)
        for i in range(hd // 2):                                     # each (i, i+hd/2) pair keeps its norm
            assert math.isclose(r[0, i] ** 2 + r[0, i + hd // 2] ** 2,
                                q[0, i] ** 2 + q[0, i + hd // 2] ** 2, rel_tol=1e-12)
    # relative-position property
    d1 = decoder.rope(q, 13, theta)[0] @ decoder.rope(k, 4, theta)[0]
    d2 = decoder.rope(q, 109, theta)[0] @ decoder.rope(k, 100, theta)[0]
    assert math.isclose(d1, d2, rel_tol=1e-10)
    # first pair rotates by exactly pos radians (frequency theta^0 = 1), last by pos*theta^(-(hd-2)/hd)
    e = np.zeros((1, hd)); e[0, 0] = 1.0
    r = decoder.rope(e, 2, theta)[0]
    assert math.isclose(r[0], math.cos(2.0)) and math.isclose(r[hd // 2], math.sin(2.0))
    e = np.zeros((1, hd)); e[0, hd // 2 - 1] = 1.0
    r = decoder.rope(e, 3, theta)[0]
    ang = 3 * theta ** (-(hd - 2) / hd)
    assert math.isclose(r[hd // 2 - 1], math.cos(ang)) and math.isclose(r[hd - 1], math.sin(ang))
    # vectorised over positions == one at a time
    qs = rng.normal(size=(5, 2, hd))
    all_at_once = decoder.rope(qs, np.arange(5), theta)
    for t in range(5):
        assert np.allclose(all_at_once[t], decoder.rope(qs[t], t, theta))


def test_silu_softmax():
    assert decoder.silu(np.array([0.0]))[0] == 0.0
    assert math.isclose(decoder.silu(np.array([1.0]))[0], 1 / (1 + math.exp(-1)))
    assert decoder.silu(np.array([-50.0]))[0] > -1e-15
    p = decoder.softmax(np.array([[1.0, 2.0, 3.0], [1000.0, 1000.0, 1000.0]]))
    assert np.allclose(p.sum(axis=1), 1)
    assert np.allclose(p[1], 1 / 3)
    assert np.allclose(p[0], np.exp([1, 2, 3]) / np.exp([1, 2, 3]).sum())


def test_attention_closed_forms():
    rng = np.random.default_rng(1)
    Hq, Hkv, hd = 4, 2, 8
    q = rng.normal(size=(Hq, hd))
    K = rng.normal(size=(1, Hkv, hd)); V = rng.normal(size=(1, Hkv, hd))
    o = decoder.attend_one(q, K, V, Hq, Hkv)                 # single key -> its V row
    for a in range(Hq):
        assert np.allclose(o[a], V[0, a // 2])
    K = np.zeros((5, Hkv, hd)); V = rng.normal(size=(5, Hkv, hd))
    o = decoder.attend_one(q, K, V, Hq, Hkv)                 # uniform scores -> mean of V
    for a in range(Hq):
        assert np.allclose(o[a], V[:, a // 2].mean(axis=0))
    # 1/sqrt(hd) scaling: two keys, scores differ by q.k/sqrt(hd)
    K = np.zeros((2, 1, hd)); K[1, 0] = q[0]
    V = np.zeros((2, 1, hd)); V[1, 0, 0] = 1.0
    o = decoder.attend_one(q[:1], K, V, 1, 1)
    sc = q[0] @ q[0] / math.sqrt(hd)
    assert math.isclose(o[0, 0], math.exp(sc) / (1 + math.exp(sc)), rel_tol=1e-12)
    # GQA with Hq == Hkv is plain multi-head attention
    K = rng.normal(size=(6, Hq, hd)); V = rng.normal(size=(6, Hq, hd))
    o = decoder.attend_one(q, K, V, Hq, Hq)
    for a in range(Hq):
        p = decoder.softmax(K[:, a] @ q[a] / math.sqrt(hd))
        assert np.allclose(o[a], p @ V[:, a])


# ---------------------------------------------------------------- scalar-loop model
def _scalar_forward(dims, wf, tokens):
    """Entry-by-entry evaluation with Python floats of the last position's logits."""
    d, Hq, Hkv, hd, F = dims.d_model, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.d_ff
    n = len(tokens)
    xs = [[float(wf["embed"][t][i]) for i in range(d)] for t in tokens]

    def norm(x, g):
        ms = sum(v * v for v in x) / len(x)
        return [v / math.sqrt(ms + dims.rms_eps) * float(gi) for v, gi in zip(x, g)]

    def matvec(W, x):
        return [sum(float(W[r][c]) * x[c] for c in range(len(x))) for r in range(len(W))]

    def rot(vec, pos):
        out = list(vec)
        for h in range(len(vec) // hd):
            for i in range(hd // 2):
                ang = pos * dims.rope_theta ** (-2.0 * i / hd)
                a, b = vec[h * hd + i], vec[h * hd + i + hd // 2]
                out[h * hd + i] = a * math.cos(ang) - b * math.sin(ang)
                out[h * hd + i + hd // 2] = b * math.cos(ang) + a * math.sin(ang)
        return out

    for l in range(dims.n_layers):
        hs = [norm(x, wf["attn_norm"][l]) for x in xs]
        qs = [rot(matvec(wf["wq"][l], h), t) for t, h in enumerate(hs)]
        ks = [rot(matvec(wf["wk"][l], h), t) for t, h in enumerate(hs)]
        vs = [matvec(wf["wv"][l], h) for h in hs]
        for t in range(n):
            o = [0.0] * (Hq * hd)
            for a in range(Hq):
                kv = a // (Hq // Hkv)
                sc = [sum(qs[t][a * hd + i] * ks[u][kv * hd + i] for i in range(hd)) / math.sqrt(hd)
                      for u in range(t + 1)]
                m = max(sc)
                e = [math.exp(v - m) for v in sc]
                Zs = sum(e)
                for i in range(hd):
                    o[a * hd + i] = sum(e[u] / Zs * vs[u][kv * hd + i] for u in range(t + 1))
            proj = matvec(wf["wo"][l], o)
            xs[t] = [a + b for a, b in zip(xs[t], proj)]
        for t in range(n):
            h2 = norm(xs[t], wf["mlp_norm"][l])
            gate = matvec(wf["w_gate"][l], h2)
            up = matvec(wf["w_up"][l], h2)
            act = [g / (1 + math.exp(-g)) * u for g, u in zip(gate, up)]
            dn = matvec(wf["w_down"][l], act)
            xs[t] = [a + b for a, b in zip(xs[t], dn)]
    return matvec(wf["lm_head"], norm(xs[-1], wf["final_norm"]))


def test_hand_sized_model_against_scalar_loops():
    shape = synth.DecoderShape("hand", 2, 8, 4, 2, 4, 6, 11, rms_eps=1e-6, rope_theta=100.0)
    bits = synth.weights_to_bits(synth.make_weights(shape, weight_seed=5, std=0.5))
    # non-trivial gains so a dropped gain shows up
    rng = np.random.default_rng(2)
    import torch
    for name in ("attn_norm", "mlp_norm"):
        bits[name] = [synth.bf16_bits(torch.tensor(rng.uniform(0.5, 1.5, size=8)).to(torch.bfloat16))
                      for _ in range(2)]
    bits["final_norm"] = synth.bf16_bits(torch.tensor(rng.uniform(0.5, 1.5, size=8)).to(torch.bfloat16))
    dims = _dims(shape)
    w = decoder.Weights(bits)
    wf = {k: ([decoder.widen_bf16(b) for b in v] if isinstance(v, list) else decoder.widen_bf16(v))
          for k, v in bits.items()}
    tokens = [3, 10, 0, 7, 7]
    want = _scalar_forward(dims, wf, tokens)
    got_c = decoder.forward_sequence(dims, w, tokens, want_from=len(tokens) - 1)[0]
    assert np.allclose(got_c, want, rtol=1e-10, atol=1e-12)
    cache = decoder.KVCache(dims.n_layers)
    for t in tokens:
        got_a = decoder.step(dims, w, t, cache)
    assert np.allclose(got_a, want, rtol=1e-10, atol=1e-12)
    assert np.abs(np.asarray(want)).max() > 0.05       # not a degenerate all-zero check


# ---------------------------------------------------------------- mode agreement on the tiny config
@pytest.fixture(scope="module")
def tiny():
    wl = synth.WORKLOADS["tiny"]
    bits = synth.weights_to_bits(synth.make_weights(wl.shape, wl.weight_seed))
    return wl, _dims(wl.shape), decoder.Weights(bits)


def test_cached_equals_recompute_equals_forced(tiny):
    wl, dims, w = tiny
    prompts = synth.make_prompts(2, 12, wl.shape.vocab, wl.prompt_seed)
    lens = [12, 9]
    G, T = 2, 5
    a = decoder.rollout_cached(dims, w, prompts, lens, G, T, 1.0, wl.sample_seed, version=7)
    b = decoder.rollout_recompute(dims, w, prompts, lens, G, T, 1.0, wl.sample_seed, version=7)
    assert np.array_equal(a.tokens, b.tokens)
    assert np.allclose(a.logprobs, b.logprobs, atol=1e-9)
    assert a.version == 7
    for p in range(2):
        for g in range(G):
            sc = decoder.score_forced(dims, w, prompts[p][:lens[p]], a.tokens[p, g], 1.0,
                                      wl.sample_seed, p * G + g)
            assert np.array_equal(sc.own_token, a.tokens[p, g])
            assert np.allclose(sc.logprob_given, a.logprobs[p, g], atol=1e-9)
            assert np.allclose(sc.margin, a.margins[p, g], atol=1e-9)
    # logits of cached decoding equal the full recompute at every step
    cache = decoder.KVCache(dims.n_layers)
    seq = [int(t) for t in prompts[0][:12]]
    for i, t in enumerate(seq):
        z = decoder.step(dims, w, t, cache)
        zf = decoder.forward_sequence(dims, w, seq[: i + 1], want_from=i)[0]
        assert np.allclose(z, zf, atol=1e-10)


def test_end_of_sequence_rule(tiny):
    """eos_id >= 0: a sequence ends at the first eos token it emits; later positions hold eos with
    log-probability 0; everything before that, and every sequence that never emits it, is unchanged
    (the noise streams do not depend on the trajectory).  Modes A, B and C agree."""
    wl, dims, w = tiny
    prompts = synth.make_prompts(2, 10, wl.shape.vocab, wl.prompt_seed)
    lens = [10, 7]
    G, T = 2, 6
    base = decoder.rollout_cached(dims, w, prompts, lens, G, T, 1.0, wl.sample_seed)
    p0, g0, j0 = 1, 0, 2
    eos = int(base.tokens[p0, g0, j0])
    a = decoder.rollout_cached(dims, w, prompts, lens, G, T, 1.0, wl.sample_seed, eos_id=eos)
    b = decoder.rollout_recompute(dims, w, prompts, lens, G, T, 1.0, wl.sample_seed, eos_id=eos)
    assert np.array_equal(a.tokens, b.tokens) and np.allclose(a.logprobs, b.logprobs, atol=1e-9)
    for p in range(2):
        for g in range(G):
            hits = np.flatnonzero(base.tokens[p, g] == eos)
            if len(hits) == 0:                      # never emitted: identical to the run without the rule
                assert np.array_equal(a.tokens[p, g], base.tokens[p, g])
                assert np.allclose(a.logprobs[p, g], base.logprobs[p, g], atol=1e-12)
                continue
            e = int(hits[0])
            assert np.array_equal(a.tokens[p, g, : e + 1], base.tokens[p, g, : e + 1])
            assert np.allclose(a.logprobs[p, g, : e + 1], base.logprobs[p, g, : e + 1], atol=1e-12)
            assert np.all(a.tokens[p, g, e + 1:] == eos) and np.all(a.logprobs[p, g, e + 1:] == 0.0)
            sc = decoder.score_forced(dims, w, prompts[p][:lens[p]], a.tokens[p, g], 1.0, wl.sample_seed,
                                      p * G + g, eos_id=eos)
            assert np.array_equal(sc.own_token, a.tokens[p, g])
            assert np.allclose(sc.logprob_given, a.logprobs[p, g], atol=1e-9)
    assert int(np.flatnonzero(base.tokens[p0, g0] == eos)[0]) <= j0 and np.all(a.tokens[p0, g0, j0 + 1:] == eos)
    # the sum of log-probabilities of a finished sequence is that of its tokens up to and including eos
    e = int(np.flatnonzero(a.tokens[p0, g0] == eos)[0])
    assert math.isclose(a.logprobs[p0, g0].sum(), base.logprobs[p0, g0, : e + 1].sum(), rel_tol=1e-12)


def test_prefix_shared_equals_per_sample_prefill(tiny):
    wl, dims, w = tiny
    prompts = synth.make_prompts(1, 10, wl.shape.vocab, 5)
    a = decoder.rollout_cached(dims, w, prompts, [10], 3, 4, 1.0, 9, share_prefix=True)
    b = decoder.rollout_cached(dims, w, prompts, [10], 3, 4, 1.0, 9, share_prefix=False)
    assert np.array_equal(a.tokens, b.tokens)
    assert np.allclose(a.logprobs, b.logprobs, atol=1e-12)
    # the G first tokens are draws from one logits row: logprobs of equal tokens coincide
    cache, z0 = decoder.prefill(dims, w, prompts[0])
    for g in range(3):
        d = sampler.draw(z0, 1.0, 9, g, 0)
        assert d.token == a.tokens[0, g, 0] and math.isclose(d.logprob, a.logprobs[0, g, 0])
    # different samples of a group really differ (streams keyed by sequence id)
    assert len({tuple(a.tokens[0, g]) for g in range(3)}) == 3


def test_layer_provider_streams_layers(tiny):
    wl, dims, w = tiny
    toks = [1, 2, 3, 4, 5, 6]
    z = decoder.forward_sequence(dims, w, toks, want_from=3)
    z2 = decoder.forward_sequence(dims, w, toks, want_from=3, layer_provider=lambda l: w.layers[l])
    assert np.array_equal(z, z2)
    assert z.shape == (3, dims.vocab)

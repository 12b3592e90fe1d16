"""The oracle's rounding diagnostic (oracle/rounding.py): where a 16-bit path loses its accuracy.

Diagnostic only: nothing here decides whether the CUDA path passes.  The tests pin the two rounding
routines to values fixed by the formats themselves, check that the instrumented forward with no
rounding IS the oracle's forward, and reproduce, on a deep narrow model that runs in seconds, the
finding the full-size GPU tests rest on: in a random-init decoder the 16-bit roundings of the FIRST
layers dominate the error of the final log-probabilities (layer 0's attention block forms the whole
residual stream that the first MLP normalises), so keeping those layers' operands in IEEE half
removes most of it.
"""
import dataclasses

import numpy as np
import pytest

from oracle import decoder, rounding
from paper_2602_02192_b200 import synth


def test_round_bf16_known_values():
    # 8-bit significand, ties to even: spacing in [1, 2) is 2^-7
    u = 2.0 ** -7
    x = np.array([1.0, 1.0 + u / 2, 1.0 + 1.5 * u, 1.0 + u / 2 + 2.0 ** -20, -(1.0 + 2.5 * u), 3.0e38, 0.0])
    want = np.array([1.0, 1.0, 1.0 + 2 * u, 1.0 + u, -(1.0 + 2 * u), 3.0e38, 0.0])
    got = rounding.round_bf16(x)
    assert np.array_equal(got[:5], want[:5]) and got[6] == 0.0
    assert abs(got[5] - 3.0e38) / 3.0e38 < 2.0 ** -8
    # every bf16 value is a fixed point; the result always fits in 16 bits of an fp32 pattern
    r = np.random.default_rng(0).normal(size=1000)
    g = rounding.round_bf16(r)
    assert np.array_equal(rounding.round_bf16(g), g)
    assert np.all(g.astype(np.float32).view(np.uint32) & 0xFFFF == 0)
    assert np.max(np.abs(g - r) / np.abs(r)) <= 2.0 ** -8


def test_round_fp16_known_values():
    # 11-bit significand: spacing in [1, 2) is 2^-10; largest finite value 65504; subnormals step 2^-24
    u = 2.0 ** -10
    x = np.array([1.0 + u / 2, 1.0 + 1.5 * u, 65504.0, 65520.0, 2.0 ** -24, 2.0 ** -25 * 1.01, 3.0 * 2.0 ** -26])
    got = rounding.round_fp16(x)
    assert got[0] == 1.0 and got[1] == 1.0 + 2 * u and got[2] == 65504.0 and np.isinf(got[3])
    assert got[4] == 2.0 ** -24 and got[5] == 2.0 ** -24 and got[6] == 2.0 ** -24
    # a bf16 value converts to half exactly when 2^-17 <= |w| <= 65504 (8 significant bits fit above 2^-24)
    w = rounding.round_bf16(np.random.default_rng(1).normal(size=4000) * 0.02)
    big = np.abs(w) >= 2.0 ** -17
    assert np.array_equal(rounding.round_fp16(w[big]), w[big])
    assert np.max(np.abs(rounding.round_fp16(w) - w)) <= 2.0 ** -25


@pytest.fixture(scope="module")
def deep_narrow():
    """12 layers, d_model 256: deep enough for the layer-0 effect, a second of numpy per plan."""
    shape = dataclasses.replace(synth.SHAPES["tiny"], n_layers=12, vocab=512)
    # N(0, 0.08^2): the same gain per matrix (std * sqrt(d_model) = 1.28) as the 8B shape has with N(0, 0.02^2)
    w = decoder.Weights(synth.weights_to_bits(synth.make_weights(shape, 0, std=0.08)))
    dims = decoder.ModelDims(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                             shape.d_ff, shape.vocab)
    toks = synth.make_prompts(1, 48, shape.vocab, 5)[0]
    return dims, w, toks


def test_no_rounding_is_the_oracle_forward(deep_narrow):
    dims, w, toks = deep_narrow
    z = rounding.forward_sequence_rounded(dims, w, toks, [rounding.Plan(())])[0]
    ref = decoder.forward_sequence(dims, w, toks)
    assert np.max(np.abs(z - ref)) < 1e-11
    lp = rounding.logprob_of_next(ref, toks)
    assert lp.shape == (len(toks) - 1,) and np.all(lp < 0)


def test_first_layers_dominate_the_16_bit_error(deep_narrow):
    dims, w, toks = deep_narrow
    P = rounding.POINTS
    L = dims.n_layers
    plans = [rounding.Plan((), name="exact"),
             rounding.Plan(P, name="bf16 everywhere"),
             rounding.Plan(P, {0: ()}, name="layer 0 exact"),
             rounding.Plan(P, {L - 1: ()}, name="last layer exact"),
             rounding.Plan(P, half_layers=range(2), name="layers 0-1 half"),
             rounding.Plan(P, half_layers=range(L + 1), name="half everywhere"),
             rounding.Plan(("k", "v"), name="only cached K/V rounded")]
    zs = rounding.forward_sequence_rounded(dims, w, toks, plans)
    ref = rounding.logprob_of_next(zs[0], toks)
    err = {p.name: float(np.mean(np.abs(rounding.logprob_of_next(z, toks) - ref))) for p, z in zip(plans, zs)}
    print({k: f"{v:.2e}" for k, v in err.items()})
    assert err["exact"] == 0.0
    # one exact layer out of twelve removes a large share if it is the first one, almost nothing if the last
    assert err["layer 0 exact"] < 0.75 * err["bf16 everywhere"]
    assert err["last layer exact"] > 0.85 * err["bf16 everywhere"]
    # half precision in two layers of twelve buys more than half of what it buys everywhere
    gain_two = err["bf16 everywhere"] - err["layers 0-1 half"]
    gain_all = err["bf16 everywhere"] - err["half everywhere"]
    assert gain_two > 0.5 * gain_all and err["half everywhere"] < 0.25 * err["bf16 everywhere"]
    # the cache alone (bf16 K/V, everything else exact) already carries a large part of the error
    assert err["only cached K/V rounded"] > 0.3 * err["bf16 everywhere"]

"""Shared pieces of the GPU parity tests: oracle-side scoring of a GPU rollout."""
import numpy as np

from oracle import decoder

LOGPROB_TOL = 5e-2        # |GPU logprob - oracle logprob| bound (fp32 accumulate, bf16 inputs)
MARGIN_EXEMPT = 1e-2      # tokens may differ only where the oracle's top-2 perturbed gap is below this


def dims_of(shape):
    return decoder.ModelDims(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads,
                             shape.head_dim, shape.d_ff, shape.vocab, shape.rms_eps, shape.rope_theta)


def check_sequences(dims, w, prompts, lens, G, temperature, seed, tokens, logprobs, seqs, steps=None,
                    layer_provider=None):
    """Teacher-forced oracle scoring along the GPU's own tokens for the given sequence ids.
    Returns (n_checked, n_exempt, max |dlogprob|).  Asserts the acceptance rule."""
    n_checked = n_exempt = 0
    worst = 0.0
    for s in seqs:
        p, g = divmod(s, G)
        sc = decoder.score_forced(dims, w, prompts[p][: int(lens[p])], tokens[p, g], temperature, seed, s,
                                  layer_provider=layer_provider, steps=steps)
        T = len(sc.own_token)
        for j in range(T):
            y = int(tokens[p, g, j])
            n_checked += 1
            if y != sc.own_token[j]:
                assert sc.margin[j] < MARGIN_EXEMPT and y == sc.runner_up[j], (
                    f"token mismatch at seq {s} step {j}: gpu {y}, oracle {sc.own_token[j]} "
                    f"(runner-up {sc.runner_up[j]}, margin {sc.margin[j]:.3e})")
                n_exempt += 1
            d = abs(float(logprobs[p, g, j]) - sc.logprob_given[j])
            worst = max(worst, d)
            assert d <= LOGPROB_TOL, f"logprob off by {d:.3e} at seq {s} step {j}"
    return n_checked, n_exempt, worst


def assert_same_rollout(tok_a, lp_a, tok_b, lp_b):
    """Two rollouts with the same seed, prompts and weights.  The split projections add their
    partial sums in memory in whatever order the CTAs finish, so logits can differ in the last
    fp32 bits between runs; a token can flip only where two perturbed scores are that close, and
    the sequence differs from there on.  Until the first flip everything must agree."""
    tok_a, tok_b = np.asarray(tok_a), np.asarray(tok_b)
    same = np.logical_and.accumulate(tok_a == tok_b, axis=-1)       # still identical up to this step
    assert same.mean() >= 0.97, same.mean()
    assert np.max(np.abs(np.asarray(lp_a) - np.asarray(lp_b))[same]) < 1e-3

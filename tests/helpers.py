"""Shared pieces of the GPU parity tests: oracle-side scoring of a GPU rollout."""
import numpy as np

from oracle import decoder

LOGPROB_TOL = 5e-2        # |GPU logprob - oracle logprob| bound (fp32 accumulate, bf16 inputs)
MARGIN_EXEMPT = 1e-2      # tokens may differ only where the oracle's top-2 perturbed gap is below this


def dims_of(shape):
    return decoder.ModelDims(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads,
                             shape.head_dim, shape.d_ff, shape.vocab, shape.rms_eps, shape.rope_theta)


def score_sequences(dims, w, prompts, lens, G, temperature, seed, tokens, logprobs, seqs, steps=None,
                    layer_provider=None):
    """Teacher-forced oracle scoring along the GPU's own tokens.  Returns per checked token:
    |dlogprob|, whether the GPU token is the oracle's own draw, whether it is the runner-up, and the
    oracle's top-2 perturbed-score margin."""
    delta, same, second, margin = [], [], [], []
    for s in seqs:
        p, g = divmod(s, G)
        sc = decoder.score_forced(dims, w, prompts[p][: int(lens[p])], tokens[p, g], temperature, seed, s,
                                  layer_provider=layer_provider, steps=steps)
        for j in range(len(sc.own_token)):
            y = int(tokens[p, g, j])
            delta.append(abs(float(logprobs[p, g, j]) - sc.logprob_given[j]))
            same.append(y == sc.own_token[j])
            second.append(y == sc.runner_up[j])
            margin.append(sc.margin[j])
    return np.asarray(delta), np.asarray(same), np.asarray(second), np.asarray(margin)


def check_sequences(dims, w, prompts, lens, G, temperature, seed, tokens, logprobs, seqs, steps=None,
                    layer_provider=None, eos_id=-1, top_p=1.0):
    """Teacher-forced oracle scoring along the GPU's own tokens for the given sequence ids.
    Returns (n_checked, n_exempt, max |dlogprob|).  Asserts the acceptance rule."""
    n_checked = n_exempt = 0
    worst = 0.0
    for s in seqs:
        p, g = divmod(s, G)
        sc = decoder.score_forced(dims, w, prompts[p][: int(lens[p])], tokens[p, g], temperature, seed, s,
                                  layer_provider=layer_provider, steps=steps, eos_id=eos_id, top_p=top_p)
        T = len(sc.own_token)
        for j in range(T):
            y = int(tokens[p, g, j])
            n_checked += 1
            if top_p < 1.0 and not np.isfinite(sc.logprob_given[j]):
                # the token sits outside the oracle's nucleus: only possible for the few ids around the
                # cut, whose place the kernel decides from fp32 mass sums (counted as exempt)
                n_exempt += 1
                continue
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
    partial sums in memory in whatever order the CTAs finish, so sums can differ in the last fp32
    bits between runs; where that flips the bf16 rounding of an activation a logit moves by ~1e-3,
    and a token can flip where two perturbed scores are that close.  The sequence differs from
    there on; until the first flip everything must agree within the log-probability bound."""
    tok_a, tok_b = np.asarray(tok_a), np.asarray(tok_b)
    same = np.logical_and.accumulate(tok_a == tok_b, axis=-1)       # still identical up to this step
    assert same.mean() >= 0.9, same.mean()
    assert np.max(np.abs(np.asarray(lp_a) - np.asarray(lp_b))[same]) < LOGPROB_TOL


class StreamedWeights:
    """Feeds the oracle one layer at a time from bf16 torch tensors (exact widening to fp64), so a
    shape whose fp64 weights would not fit in host memory can still be scored."""

    def __init__(self, weights):
        import torch
        self._t = torch
        self.w = weights
        self.lm_head = self._wide(weights["lm_head"])
        self.final_norm = self._wide(weights["final_norm"])
        self.embed = _EmbedRows(weights["embed"], self._wide)

    def _wide(self, t):
        return t.detach().to("cpu").to(self._t.float64).numpy()

    def layer(self, l):
        return {k: self._wide(self.w[k][l]) for k in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down",
                                                      "attn_norm", "mlp_norm")}


class _EmbedRows:
    def __init__(self, t, wide):
        self.t, self.wide = t, wide

    def __getitem__(self, ids):
        import torch
        idx = torch.as_tensor(np.asarray(ids), device=self.t.device, dtype=torch.long)
        return self.wide(self.t[idx])

"""Temperature sampling by Gumbel-max and the sampler's log-probability (oracle side).

What is sampled: y_t ~ pi(. | x, y_<t) at temperature T (Section 5.1 lists
temperature 1.0; Algorithm 1's rollout plane samples y ~ pi_v(.|x)).  What is
recorded: log pi_sampler(y_t | ...), the denominator of the truncated importance
ratio in the GRPO objective of Appendix F — the log-probability under exactly
the distribution that was sampled from.

  s_v     = z_v / T
  tok     = argmax_v (s_v + g_v)          ties -> lowest id
  logprob = s_tok - logsumexp(s)

Gumbel-max draws tok with probability softmax(s)_tok exactly, so no sort or
cumulative sum over the vocabulary is needed when top-p = 1.

Nucleus truncation (Section 5.1 samples with top-p 0.95): with 0 < top_p < 1 the
tokens are ranked by probability (equal probabilities: lower id first) and the
nucleus is the shortest prefix of that ranking whose probability mass reaches
top_p.  The draw is the Gumbel-argmax over the nucleus only, with the same noise
stream, and the recorded log-probability is taken under the distribution that
was actually sampled from, i.e. renormalised over the nucleus:
  logprob = s_tok - logsumexp(s_v : v in nucleus).

Pins: frequency of tokens over many seeds against softmax on a toy row
(chi-square), sum_v exp(logprob_v) = 1, logprob <= 0, tie rule, brute-force
argmax.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import philox


@dataclass
class Draw:
    token: int          # argmax of perturbed scores
    logprob: float      # log-probability of `token` under softmax(z / T)
    runner_up: int      # id with the second-largest perturbed score
    margin: float       # best - second-best perturbed score (>= 0)
    logprobs: np.ndarray  # log-probability row under the sampled distribution (fp64; -inf outside the nucleus)
    nucleus_size: int = 0     # tokens in the nucleus (the whole vocabulary when top_p = 1)
    nucleus_mass: float = 1.0  # their probability mass under softmax(z / T)


def log_softmax(s: np.ndarray) -> np.ndarray:
    s = np.asarray(s, dtype=np.float64)
    m = np.max(s)
    return s - (m + np.log(np.sum(np.exp(s - m))))


def nucleus_mask(logp: np.ndarray, top_p: float) -> np.ndarray:
    """Boolean mask of the nucleus of a log-probability row: the shortest prefix, in
    order of decreasing probability (ties: increasing id), whose mass is >= top_p."""
    if not (0.0 < top_p <= 1.0):
        raise ValueError("top_p must be in (0, 1]")
    logp = np.asarray(logp, dtype=np.float64)
    V = len(logp)
    mask = np.ones(V, dtype=bool)
    if top_p >= 1.0:
        return mask
    order = np.lexsort((np.arange(V), -logp))        # primary key: -logp; then the id
    cum = np.cumsum(np.exp(logp[order]))
    k = min(int(np.searchsorted(cum, top_p, side="left")) + 1, V)   # smallest k with cum[k-1] >= top_p
    mask[:] = False
    mask[order[:k]] = True
    return mask


def draw_with_noise(z: np.ndarray, temperature: float, g: np.ndarray, top_p: float = 1.0) -> Draw:
    """One draw given the logits row z and a Gumbel noise row g."""
    if not temperature > 0.0:
        raise ValueError("temperature must be > 0")
    s = np.asarray(z, dtype=np.float64) / float(temperature)
    lp = log_softmax(s)
    mask = nucleus_mask(lp, top_p)
    mass = float(np.sum(np.exp(lp[mask])))
    pert = np.where(mask, s + g, -np.inf)
    tok = int(np.argmax(pert))                      # np.argmax returns the first maximum
    lp = np.where(mask, lp - np.log(mass), -np.inf) if top_p < 1.0 else lp
    if int(mask.sum()) > 1:
        rest = pert.copy()
        rest[tok] = -np.inf
        ru = int(np.argmax(rest))
        margin = float(pert[tok] - rest[ru])
    else:
        ru, margin = tok, float("inf")
    return Draw(tok, float(lp[tok]), ru, margin, lp, int(mask.sum()), mass)


def draw(z: np.ndarray, temperature: float, seed: int, s: int, j: int, top_p: float = 1.0) -> Draw:
    """Draw for sequence id s at new-token index j under `seed`."""
    g = philox.gumbel_noise(seed, s, j, len(z))
    return draw_with_noise(z, temperature, g, top_p)

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
cumulative sum over the vocabulary is needed.  Nucleus truncation (top-p) is
not applied (top-p = 1).

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
    logprobs: np.ndarray  # full log-softmax row (fp64)


def log_softmax(s: np.ndarray) -> np.ndarray:
    s = np.asarray(s, dtype=np.float64)
    m = np.max(s)
    return s - (m + np.log(np.sum(np.exp(s - m))))


def draw_with_noise(z: np.ndarray, temperature: float, g: np.ndarray) -> Draw:
    """One draw given the logits row z and a Gumbel noise row g."""
    if not temperature > 0.0:
        raise ValueError("temperature must be > 0")
    s = np.asarray(z, dtype=np.float64) / float(temperature)
    pert = s + g
    tok = int(np.argmax(pert))                      # np.argmax returns the first maximum
    lp = log_softmax(s)
    if len(pert) > 1:
        rest = pert.copy()
        rest[tok] = -np.inf
        ru = int(np.argmax(rest))
        margin = float(pert[tok] - rest[ru])
    else:
        ru, margin = tok, float("inf")
    return Draw(tok, float(lp[tok]), ru, margin, lp)


def draw(z: np.ndarray, temperature: float, seed: int, s: int, j: int) -> Draw:
    """Draw for sequence id s at new-token index j under `seed`."""
    g = philox.gumbel_noise(seed, s, j, len(z))
    return draw_with_noise(z, temperature, g)

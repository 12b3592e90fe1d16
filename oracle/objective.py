"""GRPO-style clipped surrogate with truncated importance sampling (oracle side), fp64.

Appendix F, "GRPO-Style Policy Gradient Objective".  For sequence i with response
mask m_t, broadcast advantage A (one value per sequence) and per-token
log-probabilities of the taken tokens under three policies:

  rho_t  = pi_theta(y_t) / pi_theta_old(y_t)                 (likelihood ratio)
  w_t    = min( pi_learner(y_t; theta_old) / pi_sampler(y_t; theta_old), C )
                                                              (truncated importance ratio)
  term_t = min( rho_t * A, clip(rho_t, 1 - eps_c, 1 + eps_c) * A )
  J_i    = sum_t m_t * w_t * term_t / sum_t m_t

Readings (the appendix leaves them open): the truncated ratio is taken per token
(the expectation is over actions, and the ratio is written for an action a); a
sequence whose mask is empty scores 0.  The KL term beta * D_KL(pi_theta || pi_ref)
is written without an estimator; a rollout record holds log-probabilities of the
taken tokens only, so `grpo_objective` takes the per-token estimate on the taken
token that GRPO's original formulation uses,
  k_t = pi_ref(y_t) / pi_theta(y_t) - log(pi_ref(y_t) / pi_theta(y_t)) - 1  (>= 0),
whose expectation over y_t ~ pi_theta is the exact divergence, inside the same
masked mean and under the same truncated ratio as the surrogate term (the ratio
multiplies the whole of J-bar in the appendix):
  J_i = sum_t m_t * w_t * (term_t - beta * k_t) / sum_t m_t.

Pins: rho = 1 and w = 1 give J_i = A; the four clipping cases by sign of A;
the truncation caps w at C; the mask only counts response tokens; a scalar-loop
evaluation of the same formula on random inputs; k_t = 0 for equal policies, its
mean under pi_theta equals sum_v pi_theta(v) log(pi_theta(v) / pi_ref(v)) on small
categorical distributions, and with A = 0 the objective is -beta times the masked
mean of k_t.
"""
from __future__ import annotations

import numpy as np


def grpo_surrogate(logp_new, logp_old, logp_sampler, adv, mask, eps_clip: float, C: float) -> np.ndarray:
    """logp_* [n][T] (log-probabilities of the taken tokens), adv [n], mask [n][T] (0/1)
    -> J [n] (fp64)."""
    ln = np.asarray(logp_new, dtype=np.float64)
    lo = np.asarray(logp_old, dtype=np.float64)
    ls = np.asarray(logp_sampler, dtype=np.float64)
    a = np.asarray(adv, dtype=np.float64)
    m = np.asarray(mask, dtype=np.float64)
    if ln.shape != lo.shape or ln.shape != ls.shape or ln.shape != m.shape or a.shape != ln.shape[:1]:
        raise ValueError("shapes: logp_* and mask [n][T], adv [n]")
    if not (eps_clip >= 0.0) or not (C > 0.0):
        raise ValueError("eps_clip >= 0 and C > 0")
    n, T = ln.shape
    out = np.zeros(n)
    for i in range(n):
        num = 0.0
        den = 0.0
        for t in range(T):
            if m[i, t] == 0.0:
                continue
            rho = np.exp(ln[i, t] - lo[i, t])
            w = min(np.exp(lo[i, t] - ls[i, t]), C)
            clipped = min(max(rho, 1.0 - eps_clip), 1.0 + eps_clip)
            num += w * min(rho * a[i], clipped * a[i])
            den += 1.0
        out[i] = num / den if den > 0.0 else 0.0
    return out


def kl_token_estimate(logp_new, logp_ref) -> np.ndarray:
    """k = pi_ref / pi_theta - log(pi_ref / pi_theta) - 1 per taken token, from the two log-probabilities."""
    d = np.asarray(logp_ref, dtype=np.float64) - np.asarray(logp_new, dtype=np.float64)
    return np.exp(d) - d - 1.0


def grpo_objective(logp_new, logp_old, logp_sampler, logp_ref, adv, mask, eps_clip: float, C: float,
                   beta: float) -> np.ndarray:
    """The surrogate with the KL regulariser (see the header for the estimator): [n] fp64."""
    ln = np.asarray(logp_new, dtype=np.float64)
    lo = np.asarray(logp_old, dtype=np.float64)
    ls = np.asarray(logp_sampler, dtype=np.float64)
    lr = np.asarray(logp_ref, dtype=np.float64)
    a = np.asarray(adv, dtype=np.float64)
    m = np.asarray(mask, dtype=np.float64)
    if not (ln.shape == lo.shape == ls.shape == lr.shape == m.shape) or a.shape != ln.shape[:1]:
        raise ValueError("shapes: logp_* and mask [n][T], adv [n]")
    if not (eps_clip >= 0.0) or not (C > 0.0) or not (beta >= 0.0):
        raise ValueError("eps_clip >= 0, C > 0, beta >= 0")
    n, T = ln.shape
    out = np.zeros(n)
    for i in range(n):
        num = 0.0
        den = 0.0
        for t in range(T):
            if m[i, t] == 0.0:
                continue
            rho = np.exp(ln[i, t] - lo[i, t])
            w = min(np.exp(lo[i, t] - ls[i, t]), C)
            clipped = min(max(rho, 1.0 - eps_clip), 1.0 + eps_clip)
            d = lr[i, t] - ln[i, t]
            k = np.exp(d) - d - 1.0
            num += w * (min(rho * a[i], clipped * a[i]) - beta * k)
            den += 1.0
        out[i] = num / den if den > 0.0 else 0.0
    return out


def turn_mask(tokens, turn_start_id: int, shift_to_targets: bool = False) -> np.ndarray:
    """Appendix F, "Turn-Aware Masking": u_t = [x_t == turn_start], c_t = u_0 + ... + u_t (the chat-turn
    index of token t), m_t = [c_t > 1] * [c_t mod 2 == 1]: tokens of assistant turns after the system
    prompt.  tokens [n][T] -> uint8 [n][T].  shift_to_targets aligns the mask with next-token targets
    y_t = x_{t+1}: out[t] = m_{t+1}, last column 0.

    Pins: a hand-written five-turn dialogue; no turn-start token or a single one gives an empty mask;
    the mask is a function of the turn index only."""
    x = np.asarray(tokens)
    n, T = x.shape
    m = np.zeros((n, T), dtype=np.uint8)
    for i in range(n):
        c = 0
        for t in range(T):
            if x[i, t] == turn_start_id:
                c += 1
            m[i, t] = 1 if (c > 1 and c % 2 == 1) else 0
    if shift_to_targets:
        out = np.zeros_like(m)
        out[:, : T - 1] = m[:, 1:]
        return out
    return m

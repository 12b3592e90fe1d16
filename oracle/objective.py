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
(the expectation is over actions, and the ratio is written for an action a); the
KL term needs a reference policy's full distribution, which is outside this
path, so it is left out (beta = 0); a sequence whose mask is empty scores 0.

Pins: rho = 1 and w = 1 give J_i = A; the four clipping cases by sign of A;
the truncation caps w at C; the mask only counts response tokens; a scalar-loop
evaluation of the same formula on random inputs.
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

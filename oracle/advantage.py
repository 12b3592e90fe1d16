"""Group-wise reward normalisation (oracle side), fp64.

Appendix F ("group-wise normalization" equation): for the rewards R_j of one
group, A_i = (R_i - Mean(R)) / (Std(R) + eps).  The equation does not say which
standard deviation; the listing printed under it normalises with the tensor
library's default std, which divides by (n - 1), and adds eps = 1e-6 to the std
(outside the square root).  That reading is used here: unbiased std, eps added
to the std.  A group of one sample has no unbiased std and is rejected.

Pins: hand-computed groups in tests/golden/group_advantage_cases.txt, sum(A)=0,
unbiased std(A) = sigma/(sigma+eps), all-equal rewards -> zeros, invariance to
a shift of the rewards, scaling law under a positive rescale.
"""
from __future__ import annotations

import numpy as np


def group_advantage(rewards, eps: float = 1e-6) -> np.ndarray:
    """rewards [P][G] -> advantages [P][G] (fp64)."""
    r = np.asarray(rewards, dtype=np.float64)
    if r.ndim != 2:
        raise ValueError("rewards must be [P][G]")
    P, G = r.shape
    if G < 2:
        raise ValueError("a group needs at least two samples")
    out = np.empty_like(r)
    for p in range(P):
        mean = 0.0
        for g in range(G):
            mean += r[p, g]
        mean /= G
        ss = 0.0
        for g in range(G):
            ss += (r[p, g] - mean) ** 2
        std = (ss / (G - 1)) ** 0.5
        for g in range(G):
            out[p, g] = (r[p, g] - mean) / (std + eps)
    return out

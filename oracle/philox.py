"""Philox4x32-10 counter-based generator and the uniform → Gumbel map (oracle side).

Philox4x32-10 follows its published definition (Salmon, Moraes, Dror, Shaw,
"Parallel random numbers: as easy as 1, 2, 3", SC'11): ten rounds; each round
multiplies counter words 0 and 2 by two fixed 32-bit constants, keeps the high
and low halves of the 64-bit products, and mixes them with words 1 and 3 and the
two key words; the key is bumped by two Weyl constants between rounds.

The rollout sampler (the paper's "temperature 1.0" sampling of y ~ pi(.|x),
Section 5.1 and Algorithm 1's rollout-plane sampling step) does not say how
random numbers are drawn; the reading used here is:

  key      = (seed & 0xffffffff, seed >> 32)
  counter  = (v >> 2, j, s, 0)      v vocab id, j new-token index, s sequence id
  word     = output word (v & 3)
  w        = (float32(word) + 0.5f) * 2^-32   in IEEE fp32, w in (0, 1]
  E        = -log1p(-w)                       (exponential variate)
  g        = -log(E)                          (standard Gumbel variate)

Pins: the three known-answer vectors in tests/golden/philox4x32_10_kat.txt, an
independent big-integer evaluation in the tests, counter bijectivity on a small
range, moments of w, and the Gumbel-max frequency test in the sampler tests.
"""
from __future__ import annotations

import numpy as np

PHILOX_M0 = np.uint64(0xD2511F53)
PHILOX_M1 = np.uint64(0xCD9E8D57)
PHILOX_W0 = np.uint64(0x9E3779B9)
PHILOX_W1 = np.uint64(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)
_SH32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Vectorised Philox4x32-10.  All arguments broadcastable integer arrays of
    32-bit values; returns four uint32 arrays (the four output words)."""
    c0, c1, c2, c3, k0, k1 = np.broadcast_arrays(
        *[np.asarray(a, dtype=np.uint64) & _MASK32 for a in (c0, c1, c2, c3, k0, k1)])
    c0, c1, c2, c3, k0, k1 = [a.copy() for a in (c0, c1, c2, c3, k0, k1)]
    for rnd in range(10):
        p0 = PHILOX_M0 * c0            # 32x32 -> 64 bit product, exact in uint64
        p1 = PHILOX_M1 * c2
        hi0, lo0 = p0 >> _SH32, p0 & _MASK32
        hi1, lo1 = p1 >> _SH32, p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        if rnd != 9:
            k0 = (k0 + PHILOX_W0) & _MASK32
            k1 = (k1 + PHILOX_W1) & _MASK32
    return tuple(a.astype(np.uint32) for a in (c0, c1, c2, c3))


def noise_words(seed: int, s: int, j: int, vocab: int) -> np.ndarray:
    """uint32[vocab]: the Philox word assigned to each vocab id for sequence s at
    new-token index j (counter = (v>>2, j, s, 0), word v&3)."""
    nblk = (vocab + 3) // 4
    blk = np.arange(nblk, dtype=np.uint64)
    k0 = seed & 0xFFFFFFFF
    k1 = (seed >> 32) & 0xFFFFFFFF
    words = philox4x32_10(blk, j, s, 0, k0, k1)
    out = np.stack(words, axis=1).reshape(-1)       # [blk][word] -> id = 4*blk + word
    return out[:vocab]


def uniform_from_word(x: np.ndarray) -> np.ndarray:
    """w = (float32(x) + 0.5f) * 2^-32, every operation in IEEE fp32 (round to
    nearest even).  w lies in (0, 1]."""
    xf = np.asarray(x, dtype=np.uint32).astype(np.float32)       # RN-even conversion
    w = (xf + np.float32(0.5)) * np.float32(2.0 ** -32)
    return w.astype(np.float32)


def gumbel_from_uniform(w: np.ndarray) -> np.ndarray:
    """g = -log(-log1p(-w)) in fp64 from the exact fp32 w.  w == 1 gives -inf."""
    w64 = np.asarray(w, dtype=np.float64)
    with np.errstate(divide="ignore"):
        e = -np.log1p(-w64)
        g = -np.log(e)
    return g


def gumbel_noise(seed: int, s: int, j: int, vocab: int) -> np.ndarray:
    return gumbel_from_uniform(uniform_from_word(noise_words(seed, s, j, vocab)))

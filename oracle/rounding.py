"""Diagnostic only: the oracle's causal forward with bf16 rounding inserted at chosen points.

Test infrastructure, like the rest of this package.  It never decides whether a parity test
passes: the acceptance rule compares the CUDA path with the exact fp64 forward in decoder.py.
This module answers a different question: how much of the difference between a bf16 tensor-core
path and exact arithmetic is explained by WHERE values are rounded to bf16, layer by layer.

The paper states no precision for its rollout engine (Section 5.1 names the model family only);
the rounding points below are the ones a bf16 decoder has, named after the quantities of the
layer written out in decoder.py:

  h    attention-block input  rmsnorm(x) * g_attn        (input of the q, k, v projections)
  q    rotated queries
  k    rotated keys as cached
  v    values as cached
  p    softmax probabilities entering the P V product (unnormalised in a streaming kernel;
       here the normalised ones are rounded, which has the same relative error)
  o    attention output                                   (input of the output projection)
  h2   MLP-block input rmsnorm(x) * g_mlp                 (input of gate / up)
  act  silu(gate) * up                                    (input of the down projection)
  hf   final rmsnorm(x) * g_final                         (input of the lm_head)

A Plan says, for every (point, layer), whether the value is rounded there, and to which 16-bit
format: bf16 (8-bit significand) or, in the layers listed in `half_layers`, IEEE half (11-bit
significand).  Several plans can be evaluated in one pass over layer-streamed weights.
"""
from __future__ import annotations

from typing import Callable, Iterable, List, Optional, Sequence

import numpy as np

from . import decoder

POINTS = ("h", "q", "k", "v", "p", "o", "h2", "act", "hf")


def round_fp16(a: np.ndarray) -> np.ndarray:
    """fp64 -> nearest fp32 -> nearest-even IEEE half -> fp64 (overflow gives inf, as the conversion does)."""
    with np.errstate(over="ignore"):
        return np.asarray(a, dtype=np.float64).astype(np.float32).astype(np.float16).astype(np.float64)


def round_bf16(a: np.ndarray) -> np.ndarray:
    """fp64 -> nearest fp32 -> nearest-even bf16 -> fp64 (what a conversion of an fp32 register does)."""
    f = np.ascontiguousarray(a, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = ((u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)) << np.uint64(16)
    return r.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(a))


class Plan:
    """Which (point, layer) pairs are rounded.  `points`: the points rounded in ordinary layers;
    `layer_points`: {layer: points} overriding that for single layers (an empty tuple makes a layer
    exact).  Layer index n_layers stands for the final norm ('hf')."""

    def __init__(self, points: Iterable[str] = POINTS, layer_points: Optional[dict] = None, name: str = "",
                 half_layers: Iterable[int] = ()):
        self.points = frozenset(points)
        assert self.points <= set(POINTS)
        self.layer_points = {int(k): frozenset(v) for k, v in (layer_points or {}).items()}
        self.half_layers = frozenset(int(l) for l in half_layers)    # rounded to IEEE half (11-bit significand)
        self.name = name

    def on(self, point: str, layer: int) -> bool:
        return point in self.layer_points.get(layer, self.points)

    def rounder(self, layer: int):
        return round_fp16 if layer in self.half_layers else round_bf16


def _maybe(plan: Plan, point: str, layer: int, a: np.ndarray) -> np.ndarray:
    return plan.rounder(layer)(a) if plan.on(point, layer) else a


def forward_sequence_rounded(dims: decoder.ModelDims, w, tokens, plans: Sequence[Plan], want_from: int = 0,
                             layer_provider: Optional[Callable] = None) -> List[np.ndarray]:
    """decoder.forward_sequence evaluated once per plan (same weights, one pass over the layers).
    Returns one logits array [n - want_from, V] per plan."""
    tokens = np.asarray(tokens, dtype=np.int64)
    n = len(tokens)
    Hq, Hkv, hd = dims.n_q_heads, dims.n_kv_heads, dims.head_dim
    rep = Hq // Hkv
    pos = np.arange(n)
    causal = np.tril(np.ones((n, n), dtype=bool))
    xs = [np.array(w.embed[tokens], dtype=np.float64) for _ in plans]
    for l in range(dims.n_layers):
        lw = layer_provider(l) if layer_provider is not None else w.layers[l]
        for i, plan in enumerate(plans):
            x = xs[i]
            h = _maybe(plan, "h", l, decoder.rmsnorm(x, lw["attn_norm"], dims.rms_eps))
            q = decoder.rope((h @ lw["wq"].T).reshape(n, Hq, hd), pos, dims.rope_theta)
            k = decoder.rope((h @ lw["wk"].T).reshape(n, Hkv, hd), pos, dims.rope_theta)
            v = (h @ lw["wv"].T).reshape(n, Hkv, hd)
            q, k, v = _maybe(plan, "q", l, q), _maybe(plan, "k", l, k), _maybe(plan, "v", l, v)
            o = np.empty((n, Hq, hd))
            for a in range(Hq):
                kv = a // rep
                sc = np.where(causal, q[:, a, :] @ k[:, kv, :].T / np.sqrt(hd), -np.inf)
                p = decoder.softmax(sc, axis=-1)
                if plan.on("p", l):
                    # a streaming kernel rounds the unnormalised exponentials and divides by the exact
                    # sum of the unrounded ones
                    m = np.max(sc, axis=-1, keepdims=True)
                    e = np.exp(sc - m)
                    p = plan.rounder(l)(e) / np.sum(e, axis=-1, keepdims=True)
                o[:, a, :] = p @ v[:, kv, :]
            o = _maybe(plan, "o", l, o.reshape(n, Hq * hd))
            x = x + o @ lw["wo"].T
            h2 = _maybe(plan, "h2", l, decoder.rmsnorm(x, lw["mlp_norm"], dims.rms_eps))
            act = _maybe(plan, "act", l, decoder.silu(h2 @ lw["w_gate"].T) * (h2 @ lw["w_up"].T))
            xs[i] = x + act @ lw["w_down"].T
    out = []
    for i, plan in enumerate(plans):
        xf = _maybe(plan, "hf", dims.n_layers, decoder.rmsnorm(xs[i][want_from:], w.final_norm, dims.rms_eps))
        out.append(xf @ w.lm_head.T)
    return out


def logprob_of_next(z: np.ndarray, tokens, want_from: int = 0) -> np.ndarray:
    """log softmax(z[i])[tokens[want_from + i + 1]] for every row that has a next token."""
    tokens = np.asarray(tokens, dtype=np.int64)
    nxt = tokens[want_from + 1:]
    zz = z[: len(nxt)]
    m = zz.max(axis=-1)
    lse = m + np.log(np.exp(zz - m[:, None]).sum(axis=-1))
    return zz[np.arange(len(nxt)), nxt] - lse

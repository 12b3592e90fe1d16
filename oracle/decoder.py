"""Decoder-only transformer forward and GRPO rollout (oracle side), numpy fp64.

The paper's rollout plane "samples a response y ~ pi_v(.|x)" with a Qwen3-family
decoder (Section 5.1) and says nothing more about the network, so the layer
below is the standard pre-norm decoder those models use, with every choice the
paper leaves open listed in the repository's design notes:

  x   = embed[tok]
  per layer:
    h   = rmsnorm(x) * g_attn            rmsnorm(x) = x / sqrt(mean(x^2) + eps)
    q,k,v = Wq h, Wk h, Wv h             split into heads of head_dim
    q,k = rope(q, pos), rope(k, pos)     rotate-half pairing (i, i + hd/2),
                                         angle = pos * theta^(-2i/hd)
    o_a = softmax(q_a . K_{0..pos} / sqrt(hd)) V      kv head = a // (Hq/Hkv)
    x  += Wo concat_a(o_a)
    h2  = rmsnorm(x) * g_mlp
    x  += Wdown( silu(Wgate h2) * (Wup h2) )          silu(a) = a / (1 + e^-a)
  z   = Wlm (rmsnorm(x) * g_final)

No biases, no QK-norm, untied embed / lm_head.  Weights arrive as bf16 bit
patterns (uint16) and are widened exactly; all arithmetic is fp64.

Three ways of running it that must agree:
  A  KV-cached incremental decoding (one token at a time),
  B  full recompute of the whole sequence for every new token,
  C  teacher-forced scoring of a given token sequence in one causal pass.

Rollout: the prompt is prefetched once per prompt; the G samples of a group all
draw their first token from the same logits row (streams keyed by sequence id)
and then decode independently.

Pins: closed forms on hand-sized vectors (rmsnorm of a constant vector, RoPE
norm/relative-position/identity properties, single-key and uniform-score
attention, GQA == MHA when Hq == Hkv), a one-layer model evaluated entry by
entry with Python scalars in the tests, A == B == C agreement, prefix-shared ==
per-sample prefill.  The whole forward has no external implementation to compare
against in this repository (no pretrained weights, no third-party engine):
beyond those pins its parity is unpinned.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np

from . import sampler


@dataclass
class ModelDims:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e4


def widen_bf16(bits) -> np.ndarray:
    """uint16 bf16 bit patterns -> exact fp64 values."""
    b = np.asarray(bits, dtype=np.uint16)
    f32 = (b.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return f32.astype(np.float64)


class Weights:
    """Holds widened (fp64) weights.  `bits` is the dict produced by the input
    generator: global tensors by name, per-layer tensors as lists."""

    def __init__(self, bits: dict):
        self.embed = widen_bf16(bits["embed"])
        self.lm_head = widen_bf16(bits["lm_head"])
        self.final_norm = widen_bf16(bits["final_norm"])
        self.layers = []
        n_layers = len(bits["wq"])
        for l in range(n_layers):
            self.layers.append({k: widen_bf16(bits[k][l]) for k in
                                ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down",
                                 "attn_norm", "mlp_norm")})


# ----------------------------------------------------------------------------
# elementary pieces
# ----------------------------------------------------------------------------

def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """Row-wise x / sqrt(mean(x^2) + eps) * gain; x [..., d]."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(v: np.ndarray, pos, theta: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing.  v [..., n, H, hd], pos [n] (or scalar
    for a single token with v [..., H, hd])."""
    hd = v.shape[-1]
    half = hd // 2
    i = np.arange(half, dtype=np.float64)
    inv_freq = theta ** (-2.0 * i / hd)
    pos = np.asarray(pos, dtype=np.float64)
    ang = pos[..., None] * inv_freq                     # [n, half] or [half]
    c, s = np.cos(ang), np.sin(ang)
    if pos.ndim == 1:
        c, s = c[:, None, :], s[:, None, :]             # broadcast over heads
    a, b = v[..., :half], v[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(a: np.ndarray) -> np.ndarray:
    return a / (1.0 + np.exp(-a))


def softmax(s: np.ndarray, axis: int = -1) -> np.ndarray:
    m = np.max(s, axis=axis, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=axis, keepdims=True)


def attend_one(q: np.ndarray, K: np.ndarray, V: np.ndarray, n_q_heads: int,
               n_kv_heads: int) -> np.ndarray:
    """One query token against n cached keys.  q [Hq, hd]; K, V [n, Hkv, hd].
    Returns [Hq, hd]."""
    hd = q.shape[-1]
    rep = n_q_heads // n_kv_heads
    out = np.empty_like(q)
    for a in range(n_q_heads):
        kv = a // rep
        scores = K[:, kv, :] @ q[a] / np.sqrt(hd)
        p = softmax(scores)
        out[a] = p @ V[:, kv, :]
    return out


# ----------------------------------------------------------------------------
# mode A: KV-cached incremental decoding
# ----------------------------------------------------------------------------

class KVCache:
    def __init__(self, n_layers: int):
        self.K: List[List[np.ndarray]] = [[] for _ in range(n_layers)]
        self.V: List[List[np.ndarray]] = [[] for _ in range(n_layers)]

    def __len__(self):
        return len(self.K[0])

    def fork(self) -> "KVCache":
        c = KVCache(len(self.K))
        c.K = [list(k) for k in self.K]
        c.V = [list(v) for v in self.V]
        return c


def step(dims: ModelDims, w: Weights, tok: int, cache: KVCache) -> np.ndarray:
    """Feed one token at position len(cache); append its K/V; return logits z [V]."""
    pos = len(cache)
    Hq, Hkv, hd = dims.n_q_heads, dims.n_kv_heads, dims.head_dim
    x = w.embed[tok].copy()
    for l, lw in enumerate(w.layers):
        h = rmsnorm(x, lw["attn_norm"], dims.rms_eps)
        q = (lw["wq"] @ h).reshape(Hq, hd)
        k = (lw["wk"] @ h).reshape(Hkv, hd)
        v = (lw["wv"] @ h).reshape(Hkv, hd)
        q = rope(q, pos, dims.rope_theta)
        k = rope(k, pos, dims.rope_theta)
        cache.K[l].append(k)
        cache.V[l].append(v)
        K = np.stack(cache.K[l])
        V = np.stack(cache.V[l])
        o = attend_one(q, K, V, Hq, Hkv)
        x = x + lw["wo"] @ o.reshape(-1)
        h2 = rmsnorm(x, lw["mlp_norm"], dims.rms_eps)
        x = x + lw["w_down"] @ (silu(lw["w_gate"] @ h2) * (lw["w_up"] @ h2))
    return w.lm_head @ rmsnorm(x, w.final_norm, dims.rms_eps)


def prefill(dims: ModelDims, w: Weights, prompt) -> (KVCache, np.ndarray):
    """Run the prompt token by token; return its cache and the last logits row."""
    cache = KVCache(dims.n_layers)
    z = None
    for t in prompt:
        z = step(dims, w, int(t), cache)
    return cache, z


# ----------------------------------------------------------------------------
# modes B / C: whole-sequence causal forward
# ----------------------------------------------------------------------------

def layer_sequence(dims: ModelDims, lw: dict, x: np.ndarray) -> np.ndarray:
    """One decoder layer over a whole sequence, causal: x [n, d] (row t = position t) -> x [n, d].
    The attention block and the MLP block of the module docstring, each added to x."""
    n = x.shape[0]
    Hq, Hkv, hd = dims.n_q_heads, dims.n_kv_heads, dims.head_dim
    rep = Hq // Hkv
    pos = np.arange(n)
    causal = np.tril(np.ones((n, n), dtype=bool))
    h = rmsnorm(x, lw["attn_norm"], dims.rms_eps)
    q = (h @ lw["wq"].T).reshape(n, Hq, hd)
    k = (h @ lw["wk"].T).reshape(n, Hkv, hd)
    v = (h @ lw["wv"].T).reshape(n, Hkv, hd)
    q = rope(q, pos, dims.rope_theta)
    k = rope(k, pos, dims.rope_theta)
    o = np.empty((n, Hq, hd))
    for a in range(Hq):
        kv = a // rep
        sc = q[:, a, :] @ k[:, kv, :].T / np.sqrt(hd)         # [n, n]
        sc = np.where(causal, sc, -np.inf)
        o[:, a, :] = softmax(sc, axis=-1) @ v[:, kv, :]
    x = x + o.reshape(n, Hq * hd) @ lw["wo"].T
    h2 = rmsnorm(x, lw["mlp_norm"], dims.rms_eps)
    return x + (silu(h2 @ lw["w_gate"].T) * (h2 @ lw["w_up"].T)) @ lw["w_down"].T


def forward_sequence(dims: ModelDims, w: Weights, tokens, want_from: int = 0,
                     layer_provider=None) -> np.ndarray:
    """Causal forward over a whole sequence; logits for positions >= want_from,
    shape [n - want_from, V].  Row i predicts the token at position want_from+i+1.

    layer_provider, if given, is a callable l -> layer dict (fp64), used instead of
    w.layers so that a large model can be streamed one layer at a time."""
    tokens = np.asarray(tokens, dtype=np.int64)
    x = w.embed[tokens].copy()                                    # [n, d]
    for l in range(dims.n_layers):
        lw = layer_provider(l) if layer_provider is not None else w.layers[l]
        x = layer_sequence(dims, lw, x)
    xf = rmsnorm(x[want_from:], w.final_norm, dims.rms_eps)
    return xf @ w.lm_head.T


# ----------------------------------------------------------------------------
# rollouts
# ----------------------------------------------------------------------------

@dataclass
class Rollout:
    tokens: np.ndarray      # int32 [P][G][T]
    logprobs: np.ndarray    # fp64  [P][G][T]
    margins: np.ndarray     # fp64  [P][G][T]  top-2 perturbed-score gap
    runner_up: np.ndarray   # int32 [P][G][T]
    version: int


def _finish(toks, lps, mg, ru, p, g, j, eos_id):
    """End-of-sequence rule: a sequence that has emitted eos_id is finished; every
    later position holds eos_id with log-probability 0 (it is not sampled, so it
    contributes nothing to a sum of log-probabilities) and an infinite margin."""
    toks[p, g, j + 1:] = eos_id
    lps[p, g, j + 1:] = 0.0
    mg[p, g, j + 1:] = np.inf
    ru[p, g, j + 1:] = eos_id


def rollout_cached(dims, w, prompts, prompt_lens, G, T, temperature, seed,
                   version: int = 0, share_prefix: bool = True, eos_id: int = -1,
                   top_p: float = 1.0) -> Rollout:
    """Mode A.  share_prefix=False prefills every sample on its own (used to pin
    prefix sharing).  eos_id >= 0 enables the end-of-sequence rule (Section 5.1
    generates up to a maximum length: responses end earlier at the end token)."""
    P = len(prompts)
    toks = np.zeros((P, G, T), dtype=np.int32)
    lps = np.zeros((P, G, T))
    mg = np.zeros((P, G, T))
    ru = np.zeros((P, G, T), dtype=np.int32)
    for p in range(P):
        prompt = prompts[p][: int(prompt_lens[p])]
        if share_prefix:
            base_cache, z0 = prefill(dims, w, prompt)
        for g in range(G):
            s = p * G + g
            if share_prefix:
                cache, z = base_cache.fork(), z0
            else:
                cache, z = prefill(dims, w, prompt)
            for j in range(T):
                d = sampler.draw(z, temperature, seed, s, j, top_p)
                toks[p, g, j], lps[p, g, j], mg[p, g, j], ru[p, g, j] = \
                    d.token, d.logprob, d.margin, d.runner_up
                if eos_id >= 0 and d.token == eos_id:
                    _finish(toks, lps, mg, ru, p, g, j, eos_id)
                    break
                if j + 1 < T:
                    z = step(dims, w, d.token, cache)
    return Rollout(toks, lps, mg, ru, version)


def rollout_recompute(dims, w, prompts, prompt_lens, G, T, temperature, seed,
                      version: int = 0, eos_id: int = -1, top_p: float = 1.0) -> Rollout:
    """Mode B: the whole sequence is recomputed for every new token."""
    P = len(prompts)
    toks = np.zeros((P, G, T), dtype=np.int32)
    lps = np.zeros((P, G, T))
    mg = np.zeros((P, G, T))
    ru = np.zeros((P, G, T), dtype=np.int32)
    for p in range(P):
        prompt = [int(t) for t in prompts[p][: int(prompt_lens[p])]]
        for g in range(G):
            s = p * G + g
            seq = list(prompt)
            for j in range(T):
                z = forward_sequence(dims, w, seq, want_from=len(seq) - 1)[0]
                d = sampler.draw(z, temperature, seed, s, j, top_p)
                toks[p, g, j], lps[p, g, j], mg[p, g, j], ru[p, g, j] = \
                    d.token, d.logprob, d.margin, d.runner_up
                if eos_id >= 0 and d.token == eos_id:
                    _finish(toks, lps, mg, ru, p, g, j, eos_id)
                    break
                seq.append(d.token)
    return Rollout(toks, lps, mg, ru, version)


@dataclass
class Scored:
    logprob_given: np.ndarray   # fp64 [T]  log-prob of the given token at each step
    own_token: np.ndarray       # int32 [T] the oracle's own Gumbel-argmax
    own_logprob: np.ndarray     # fp64 [T]
    runner_up: np.ndarray       # int32 [T]
    margin: np.ndarray          # fp64 [T]


def score_forced(dims, w, prompt, given_tokens, temperature, seed, s,
                 layer_provider=None, steps: Optional[int] = None, eos_id: int = -1,
                 top_p: float = 1.0) -> Scored:
    """Mode C: teacher-forced along `given_tokens` (the T tokens some other
    implementation produced for sequence id s).  At step j the context is the
    prompt plus given_tokens[:j]; returns the log-prob of given_tokens[j] and the
    oracle's own draw for (s, j).  `steps` limits scoring to the first few steps."""
    prompt = [int(t) for t in prompt]
    given = [int(t) for t in given_tokens]
    T = len(given) if steps is None else min(steps, len(given))
    seq = prompt + given[: T - 1]
    z = forward_sequence(dims, w, seq, want_from=len(prompt) - 1, layer_provider=layer_provider)
    out = Scored(np.zeros(T), np.zeros(T, dtype=np.int32), np.zeros(T),
                 np.zeros(T, dtype=np.int32), np.zeros(T))
    finished = False                 # the GIVEN tokens decide where the sequence ends
    for j in range(T):
        if finished:
            out.logprob_given[j], out.own_token[j], out.own_logprob[j] = 0.0, eos_id, 0.0
            out.runner_up[j], out.margin[j] = eos_id, np.inf
            continue
        d = sampler.draw(z[j], temperature, seed, s, j, top_p)
        out.logprob_given[j] = d.logprobs[given[j]]
        out.own_token[j], out.own_logprob[j] = d.token, d.logprob
        out.runner_up[j], out.margin[j] = d.runner_up, d.margin
        finished = eos_id >= 0 and given[j] == eos_id
    return out

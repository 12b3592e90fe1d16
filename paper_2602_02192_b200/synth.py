"""Seeded synthetic inputs: decoder shapes, random-init weights, prompts, rewards.

This module only *generates inputs*.  It holds none of the method's arithmetic
(no normalisation, attention, sampling, paging or advantage code) and imports
neither the CUDA binding nor the CPU oracle, so both can be fed from it.

Weights are drawn per tensor from N(0, 0.02^2) in fp32 and rounded to bf16; the
bf16 *bit patterns* are what both consumers receive.  Each tensor has its own
seed, derived from (weight_seed, layer, tensor id), so a single tensor of a large
shape can be regenerated alone.  RMSNorm gains are 1.0 (a N(0, 0.02) gain would
zero the network).  Token ids are uniform in [0, vocab); rewards uniform in [0, 1).
"""
from __future__ import annotations

from dataclasses import dataclass, asdict
from typing import Dict, List

import numpy as np
import torch


@dataclass(frozen=True)
class DecoderShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e4

    def n_params(self) -> int:
        attn = self.d_model * self.head_dim * (2 * self.n_q_heads + 2 * self.n_kv_heads)
        mlp = 3 * self.d_model * self.d_ff
        return self.n_layers * (attn + mlp) + 2 * self.vocab * self.d_model

    def as_dict(self) -> dict:
        return asdict(self)


@dataclass(frozen=True)
class Workload:
    name: str
    shape: DecoderShape
    n_prompts: int
    G: int
    prompt_len: int
    new_tokens: int
    temperature: float = 1.0
    page_size: int = 16
    prompt_seed: int = 1000
    weight_seed: int = 0
    sample_seed: int = 42
    half_layers: int = 0      # leading layers whose 16-bit operands are IEEE half (engine configuration)


SHAPES: Dict[str, DecoderShape] = {
    "tiny": DecoderShape("tiny", 2, 256, 4, 2, 64, 688, 4096),
    "0.6B": DecoderShape("0.6B", 28, 1024, 16, 8, 128, 3072, 151936),
    "4B": DecoderShape("4B", 36, 2560, 32, 8, 128, 9728, 151936),
    "8B": DecoderShape("8B", 36, 4096, 32, 8, 128, 12288, 151936),
    "32B": DecoderShape("32B", 64, 5120, 64, 8, 128, 25600, 151936),
}

WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", SHAPES["tiny"], 4, 4, 32, 32, prompt_seed=1001),
    "0.6B": Workload("0.6B", SHAPES["0.6B"], 64, 8, 256, 1024, prompt_seed=1002),
    "4B": Workload("4B", SHAPES["4B"], 32, 8, 512, 2048, prompt_seed=1003, half_layers=4),
    "8B": Workload("8B", SHAPES["8B"], 32, 8, 512, 2048, prompt_seed=1004, half_layers=8),
    "32B": Workload("32B", SHAPES["32B"], 16, 8, 1024, 2048, prompt_seed=1005, half_layers=16),
}

# Tensor ids used in the per-tensor seed.  Layer index -1 is "not in a layer".
_TENSOR_IDS = {
    "embed": 0, "lm_head": 1, "final_norm": 2,
    "wq": 3, "wk": 4, "wv": 5, "wo": 6,
    "w_gate": 7, "w_up": 8, "w_down": 9,
    "attn_norm": 10, "mlp_norm": 11,
}
LAYER_TENSORS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "attn_norm", "mlp_norm")
GLOBAL_TENSORS = ("embed", "lm_head", "final_norm")


def tensor_shape(shape: DecoderShape, name: str):
    d, hd = shape.d_model, shape.head_dim
    return {
        "embed": (shape.vocab, d), "lm_head": (shape.vocab, d), "final_norm": (d,),
        "wq": (shape.n_q_heads * hd, d), "wk": (shape.n_kv_heads * hd, d),
        "wv": (shape.n_kv_heads * hd, d), "wo": (d, shape.n_q_heads * hd),
        "w_gate": (shape.d_ff, d), "w_up": (shape.d_ff, d), "w_down": (d, shape.d_ff),
        "attn_norm": (d,), "mlp_norm": (d,),
    }[name]


def tensor_seed(weight_seed: int, layer: int, name: str) -> int:
    return (int(weight_seed) * 1_000_003 + (layer + 1) * 101 + _TENSOR_IDS[name]) & 0x7FFFFFFF


def make_tensor(shape: DecoderShape, name: str, layer: int, weight_seed: int,
                device: str = "cpu", std: float = 0.02) -> torch.Tensor:
    """One weight tensor as torch.bfloat16 on `device` (row-major [out, in])."""
    dims = tensor_shape(shape, name)
    if name.endswith("norm"):
        return torch.ones(dims, dtype=torch.bfloat16, device=device)
    gen = torch.Generator(device=device)
    gen.manual_seed(tensor_seed(weight_seed, layer, name))
    out = torch.empty(dims, dtype=torch.bfloat16, device=device)
    rows_per_chunk = max(1, (1 << 26) // max(1, dims[-1]))
    for r0 in range(0, dims[0], rows_per_chunk):
        r1 = min(dims[0], r0 + rows_per_chunk)
        blk = torch.empty((r1 - r0,) + tuple(dims[1:]), dtype=torch.float32, device=device)
        blk.normal_(0.0, std, generator=gen)
        out[r0:r1] = blk.to(torch.bfloat16)
    return out


def make_weights(shape: DecoderShape, weight_seed: int = 0, device: str = "cpu",
                 std: float = 0.02) -> dict:
    """All tensors of a decoder: {'embed','lm_head','final_norm'} → tensor and the
    per-layer names → list of tensors."""
    w = {n: make_tensor(shape, n, -1, weight_seed, device, std) for n in GLOBAL_TENSORS}
    for n in LAYER_TENSORS:
        w[n] = [make_tensor(shape, n, l, weight_seed, device, std) for l in range(shape.n_layers)]
    return w


def make_weights_pinned(shape: DecoderShape, weight_seed: int = 0, gen_device: str = "cuda",
                        std: float = 0.02) -> dict:
    """Same tensors as make_weights(device=gen_device), generated one at a time on gen_device and
    kept in page-locked host memory: for shapes whose snapshot must not take device memory twice."""
    def one(name, layer):
        t = make_tensor(shape, name, layer, weight_seed, gen_device, std)
        host = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
        host.copy_(t)
        return host
    w = {n: one(n, -1) for n in GLOBAL_TENSORS}
    for n in LAYER_TENSORS:
        w[n] = [one(n, l) for l in range(shape.n_layers)]
    return w


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor → numpy uint16 array of its bit patterns (on the host)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def weights_to_bits(w: dict) -> dict:
    out = {}
    for k, v in w.items():
        out[k] = [bf16_bits(t) for t in v] if isinstance(v, list) else bf16_bits(v)
    return out


def make_prompts(n_prompts: int, prompt_len: int, vocab: int, seed: int) -> np.ndarray:
    """int32 [n_prompts][prompt_len], ids uniform in [0, vocab)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(0, vocab, size=(n_prompts, prompt_len), dtype=np.int64).astype(np.int32)


def make_ragged_prompts(lens: List[int], vocab: int, seed: int, pad_to: int | None = None):
    """Prompts of the given lengths, right-padded with zeros to a common width."""
    width = pad_to or max(lens)
    rng = np.random.Generator(np.random.PCG64(seed))
    out = np.zeros((len(lens), width), dtype=np.int32)
    for i, n in enumerate(lens):
        out[i, :n] = rng.integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)
    return out, np.asarray(lens, dtype=np.int32)


def make_rewards(n_prompts: int, G: int, seed: int) -> np.ndarray:
    """float32 [n_prompts][G], uniform in [0, 1)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.random(size=(n_prompts, G), dtype=np.float32)

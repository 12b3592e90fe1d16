"""Snapshot dissemination along forwarding chains (Section 4.3, "Peer-to-Peer Broadcast"; Appendix C.3).

The paper's learner streams a new policy snapshot to N_ch = floor(B0 / Bw) first-hop seeds; every
worker forwards each chunk to its single downstream child as soon as it has it (store and forward,
fan-out 1) and switches its local version only when the whole snapshot is installed.  Inside one node
the same scheme moves a snapshot from the rank that holds it to the rollout replicas over
torch.distributed point-to-point transfers (NCCL over NVLink between GPUs, gloo between CPU
processes): the source's outgoing link carries the snapshot N_ch times instead of once per replica,
and every replica both receives and sends at link rate.

This module is plumbing: it moves bytes and calls no kernel.  The chain plan comes from the library's
echo_chain_assemble (scores from echo_peer_score); the received tensors are installed with
Engine.echo_load_policy, which copies them into the inactive weight buffer while generation continues
on the old version.  A received chunk always lands in this rank's own memory before anything reads it.
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch
import torch.distributed as dist

GLOBAL_TENSORS = ("embed", "lm_head", "final_norm")
LAYER_TENSORS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "attn_norm", "mlp_norm")
_ALIGN = 256


def plan_chains(scores: Sequence[float], B0: float, Bw: float) -> List[List[int]]:
    """Chains of worker indices, seed first (echo_chain_assemble): N_ch = floor(B0 / Bw) chains, the best
    scored workers seed them, the rest are appended to the tails round-robin in rank order."""
    from . import binding
    n = len(scores)
    if n == 0:
        return []
    sc = np.ascontiguousarray(np.asarray(scores, dtype=np.float64))
    chain_of = (C.c_int32 * n)()
    hop_of = (C.c_int32 * n)()
    n_ch = C.c_int32()
    rc = binding.lib.echo_chain_assemble(sc.ctypes.data_as(C.POINTER(C.c_double)), n, float(B0), float(Bw),
                                         chain_of, hop_of, C.byref(n_ch))
    if rc != 0:
        raise binding.EchoError(rc)
    chains: List[List[Optional[int]]] = [[] for _ in range(n_ch.value)]
    for w in range(n):
        c, h = chain_of[w], hop_of[w]
        while len(chains[c]) <= h:
            chains[c].append(None)
        chains[c][h] = w
    return [[w for w in c if w is not None] for c in chains]


def excise(chains: List[List[int]], failed: int) -> List[List[int]]:
    """Chain repair after a relay failure (Section 4.3; Appendix D): the failed worker is cut out and its
    downstream tail is reattached to the nearest healthy parent, i.e. the chain closes over the gap."""
    return [[w for w in c if w != failed] for c in chains if any(w != failed for w in c)]


def snapshot_layout(shape) -> (List[tuple], int):
    """[(name, layer or -1, byte offset, tensor shape)] of every tensor of a snapshot in its flat byte
    buffer (bf16, 256-byte aligned), and the buffer's size.  Every rank derives it from the decoder shape."""
    from . import synth
    entries, off = [], 0
    def add(name, layer):
        nonlocal off
        dims = synth.tensor_shape(shape, name)
        entries.append((name, layer, off, dims))
        off += (int(np.prod(dims)) * 2 + _ALIGN - 1) // _ALIGN * _ALIGN
    for n in GLOBAL_TENSORS:
        add(n, -1)
    for l in range(shape.n_layers):
        for n in LAYER_TENSORS:
            add(n, l)
    return entries, off


def pack(weights: Dict, shape, device=None) -> torch.Tensor:
    """Snapshot dict -> flat uint8 buffer in snapshot_layout order."""
    entries, total = snapshot_layout(shape)
    ref = weights["embed"]
    flat = torch.zeros(total, dtype=torch.uint8, device=device if device is not None else ref.device)
    for name, layer, off, dims in entries:
        t = weights[name] if layer < 0 else weights[name][layer]
        assert t.dtype == torch.bfloat16 and tuple(t.shape) == tuple(dims)
        nbytes = t.numel() * 2
        flat[off: off + nbytes].copy_(t.contiguous().view(torch.uint8).reshape(-1))
    return flat


def unpack(flat: torch.Tensor, shape) -> Dict:
    """Views of the flat buffer as the snapshot dict echo_load_policy takes (no copy)."""
    entries, total = snapshot_layout(shape)
    assert flat.dtype == torch.uint8 and flat.numel() == total
    out: Dict = {n: [None] * shape.n_layers for n in LAYER_TENSORS}
    for name, layer, off, dims in entries:
        t = flat[off: off + int(np.prod(dims)) * 2].view(torch.bfloat16).reshape(dims)
        if layer < 0:
            out[name] = t
        else:
            out[name][layer] = t
    return out


def disseminate(flat: Optional[torch.Tensor], version: int, shape, src_rank: int, chains: List[List[int]],
                chunk_bytes: int = 8 << 20, group=None, device=None):
    """Collective over the ranks named in `chains` plus `src_rank`: the snapshot `flat` (on src_rank; None
    elsewhere) reaches every rank of every chain by chunked store-and-forward.  Returns (flat, version) on
    every participating rank; ranks outside the chains and other than the source return (None, None).

    Each chain member receives chunk k from its parent (the source for a seed), forwards it to its child
    at once, and meanwhile already receives chunk k + 1.  A rank reports the new version only after its
    last chunk has arrived: the caller installs then, and its trajectories switch version at the next
    rollout boundary."""
    rank = dist.get_rank(group)
    _, total = snapshot_layout(shape)
    n_chunks = (total + chunk_bytes - 1) // chunk_bytes
    spans = [(k * chunk_bytes, min(total, (k + 1) * chunk_bytes)) for k in range(n_chunks)]
    header = torch.zeros(2, dtype=torch.int64, device=device)

    if rank == src_rank:
        assert flat is not None and flat.numel() == total
        header[0], header[1] = int(version), total
        pending = []
        for chain in chains:
            if chain:
                pending.append(dist.isend(header, chain[0], group=group))
        for lo, hi in spans:                                   # chunk-major: every chain advances together
            for chain in chains:
                if chain:
                    pending.append(dist.isend(flat[lo:hi], chain[0], group=group))
        for req in pending:
            req.wait()
        return flat, int(version)

    mine = [(c, c.index(rank)) for c in chains if rank in c]
    if not mine:
        return None, None
    chain, hop = mine[0]
    parent = src_rank if hop == 0 else chain[hop - 1]
    child = chain[hop + 1] if hop + 1 < len(chain) else None
    buf = torch.empty(total, dtype=torch.uint8, device=device)
    dist.recv(header, parent, group=group)
    if int(header[1]) != total:
        raise RuntimeError(f"snapshot of {int(header[1])} bytes does not match this rank's shape ({total})")
    sends = []
    if child is not None:
        sends.append(dist.isend(header.clone(), child, group=group))
    nxt = dist.irecv(buf[spans[0][0]: spans[0][1]], parent, group=group)
    for k, (lo, hi) in enumerate(spans):
        nxt.wait()                                             # chunk k is complete in this rank's memory
        if k + 1 < n_chunks:
            nxt = dist.irecv(buf[spans[k + 1][0]: spans[k + 1][1]], parent, group=group)
        if child is not None:
            sends.append(dist.isend(buf[lo:hi], child, group=group))     # forward at once
    for req in sends:
        req.wait()
    return buf, int(header[0])

"""Paged KV-cache plan with one shared prompt prefix per group (oracle side).

The paper's rollout plane produces G completions per prompt (the rollout
multiplicity n of Section 5.1); it does not describe a KV cache.  The plan below
is the reading this repository uses; it is integer-only and must match the CUDA
side bit for bit.

  page size                  Z tokens (16)
  sequence id                s = p*G + g
  prompt p, length Lp[p]     full prefix pages  f_p = Lp[p] // Z
                             prefix pages       n_pre_p = ceil(Lp[p] / Z)
  new tokens T               the token fed at the last step (position Lp+T-2)
                             needs a slot, the last sampled token does not:
                             decode pages n_dec_p = ceil((Lp[p]+T-1)/Z) - f_p
  physical ids               prefix pages of prompt p:  pre_base[p] + [0, n_pre_p)
                             decode pages of sequence s: dec_base[s] + [0, n_dec_p)
                             with pre_base the running sum of n_pre over prompts
                             and dec_base continuing after all prefix pages, in
                             sequence-id order.
  logical page q of s        q <  f_p : pre_base[p] + q   (shared by the group)
                             q >= f_p : dec_base[s] + (q - f_p)
  position t                 slot (page_table[s][t // Z], t % Z)

If Lp[p] is not a multiple of Z, the prompt's partial last page is written to
pre_base[p] + f_p during prefill and then copied into the first decode page of
each of the G samples, which continue to fill it on their own.

Pins: brute-force uniqueness/sharing checks in the tests (every (s, t) maps to
one slot, no two sequences share a slot at t >= f_p*Z, all G samples share the
slots below f_p*Z), and the closed-form counts for the benchmark configs.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class PagePlan:
    page_size: int
    n_pages: int                 # total physical pages used
    width: int                   # logical pages per row of the table
    table: np.ndarray            # int32 [P*G][width], -1 where unused
    prefill_table: np.ndarray    # int32 [P][width]: where prompt p's own prefill writes
    pre_base: np.ndarray         # int32 [P]
    dec_base: np.ndarray         # int32 [P*G]
    full_prefix_pages: np.ndarray  # int32 [P]


def ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def build(prompt_lens, G: int, T: int, page_size: int = 16) -> PagePlan:
    lens = [int(x) for x in prompt_lens]
    P = len(lens)
    Z = page_size
    f = [L // Z for L in lens]
    n_pre = [ceil_div(L, Z) for L in lens]
    n_dec = [ceil_div(L + T - 1, Z) - fp for L, fp in zip(lens, f)]
    width = max(ceil_div(L + T - 1, Z) for L in lens) if P else 0
    width = max([width] + n_pre)
    pre_base = np.zeros(P, dtype=np.int32)
    acc = 0
    for p in range(P):
        pre_base[p] = acc
        acc += n_pre[p]
    dec_base = np.zeros(P * G, dtype=np.int32)
    for p in range(P):
        for g in range(G):
            dec_base[p * G + g] = acc
            acc += n_dec[p]
    table = -np.ones((P * G, width), dtype=np.int32)
    prefill_table = -np.ones((P, width), dtype=np.int32)
    for p in range(P):
        for q in range(n_pre[p]):
            prefill_table[p, q] = pre_base[p] + q
        for g in range(G):
            s = p * G + g
            for q in range(f[p] + n_dec[p]):
                table[s, q] = pre_base[p] + q if q < f[p] else dec_base[s] + (q - f[p])
    return PagePlan(Z, acc, width, table, prefill_table, pre_base, dec_base,
                    np.asarray(f, dtype=np.int32))


def slot(plan: PagePlan, s: int, t: int):
    """(physical page, offset in page) of position t of sequence s."""
    return int(plan.table[s, t // plan.page_size]), t % plan.page_size

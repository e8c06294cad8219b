"""Brute-force attention for hand-sized inputs: pure Python loops over lists of
floats, ``math.exp`` on the raw scores (no maximum subtracted), one query row
against contiguous K and V.  It exists only to pin ``attn_oracle.c`` on tiny
cases; it is a second, independently written statement of
``softmax(q K^T / sqrt(d)) V`` (the decode self-attention counted by the
paper's T_compute^d term, Section IV-C).

TEST INFRASTRUCTURE ONLY.
"""
from __future__ import annotations

import math
from typing import List, Sequence


def attn_row(q: Sequence[float], K: Sequence[Sequence[float]],
             V: Sequence[Sequence[float]]) -> List[float]:
    """q: d floats; K, V: n rows of d floats.  Returns d floats."""
    d = len(q)
    n = len(K)
    e = []
    for i in range(n):
        dot = 0.0
        for j in range(d):
            dot += float(q[j]) * float(K[i][j])
        e.append(math.exp(dot / math.sqrt(d)))
    total = 0.0
    for x in e:
        total += x
    out = []
    for j in range(d):
        acc = 0.0
        for i in range(n):
            acc += (e[i] / total) * float(V[i][j])
        out.append(acc)
    return out


def attn_batch(q, K_list, V_list, Hq: int, Hkv: int):
    """q[s][h][j]; K_list[s][i][g][j]; consecutive query heads share KV head
    g = h // (Hq // Hkv).  Returns out[s][h][j] as nested lists."""
    G = Hq // Hkv
    out = []
    for s in range(len(q)):
        per_head = []
        for h in range(Hq):
            g = h // G
            Kg = [[float(x) for x in K_list[s][i][g]] for i in range(len(K_list[s]))]
            Vg = [[float(x) for x in V_list[s][i][g]] for i in range(len(V_list[s]))]
            per_head.append(attn_row([float(x) for x in q[s][h]], Kg, Vg))
        out.append(per_head)
    return out

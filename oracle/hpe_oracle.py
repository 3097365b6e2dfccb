"""Plain fp64 definition of the hierarchical positional encoding.  TEST INFRASTRUCTURE ONLY.

Paper, paragraph "Hierarchical Positional Encoding" and its equation: a token has one index p^l
per hierarchy level l = 1..L and
    HPE(p, 2k) = sum_l sin(w_k p^l),   HPE(p, 2k+1) = sum_l cos(w_k p^l),   w_k = 10000^(-2k/d_model).
Reading of the (stripped) index figure: p^l is the number, counted from 1, of the token's level-l
ancestor (the token itself at its own level) among its siblings; levels deeper than the token's own
carry 0, the root carries 0 everywhere.  Under this numbering the paper's per-level mask equations
reproduce the parent / sibling / child rule (pinned in tests/test_oracle_pins.py).
PAD tokens get an all-zero encoding.  Shares no code with the CUDA path.
"""
from __future__ import annotations

import numpy as np


def pvectors(level, parent, cu, n_levels: int) -> np.ndarray:
    """int64 [T, n_levels]: p^1..p^L of every token (plain loops)."""
    level = np.asarray(level); parent = np.asarray(parent); cu = np.asarray(cu)
    T = len(level)
    rank = np.zeros(T, np.int64)
    for b in range(len(cu) - 1):
        s0, s1 = int(cu[b]), int(cu[b + 1])
        seen = {}                                   # parent -> children met so far
        for i in range(s0, s1):
            if level[i] < 0 or parent[i] < 0:
                continue
            p = s0 + int(parent[i])
            seen[p] = seen.get(p, 0) + 1
            rank[i] = seen[p]
    P = np.zeros((T, n_levels), np.int64)
    for b in range(len(cu) - 1):
        s0, s1 = int(cu[b]), int(cu[b + 1])
        for i in range(s0, s1):
            node, lv = i, int(level[i])
            while lv >= 1:
                if lv <= n_levels:
                    P[i, lv - 1] = rank[node]
                node = s0 + int(parent[node])
                lv -= 1
    return P


def hpe(level, parent, cu, d_model: int, n_levels: int = 3) -> np.ndarray:
    """fp64 [T, d_model]."""
    P = pvectors(level, parent, cu, n_levels).astype(np.float64)
    k = np.arange(d_model // 2, dtype=np.float64)
    w = 1.0 / np.power(10000.0, 2.0 * k / d_model)
    ang = P[:, :, None] * w[None, None, :]          # [T, L, d/2]
    out = np.zeros((len(level), d_model), np.float64)
    out[:, 0::2] = np.sin(ang).sum(1)
    out[:, 1::2] = np.cos(ang).sum(1)
    out[np.asarray(level) < 0] = 0.0
    return out

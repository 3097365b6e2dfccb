"""Plain fp64 definition of decoder cross-attention to a level subset of the encoder tokens.
TEST INFRASTRUCTURE ONLY.

Paper, paragraph "Results on FacetSum (Encoder-Decoder Models)" and the decoder of the paragraph
"Hierarchical Encoder and Decoder Stacks": the decoder's cross-attention sub-layer looks at the
encoder output of the same document, either at all tokens or only at a subset chosen by
hierarchy level ([SEC] anchors; [SEC] and [SENT] anchors; anchors and regular tokens).  Within the
chosen subset it is ordinary softmax attention:
    A = Qd Ks^T * scale,  S = softmax(A) row-wise,  O = S Vs,  LSE_i = log sum_j exp(A_ij),
where Ks, Vs are the rows of K, V whose token level has its bit set in `level_mask` (bit l = level
l; PAD tokens, level -1, are never chosen).  A decoder row of a document without a chosen token
gets O = 0, LSE = -inf and no gradient.  Backward is the derivative of that map; encoder tokens
outside the subset get zero dK, dV.

Layouts: qd, o, do, dq are [Tq, H, d] with the decoder rows of sequence b at cu_q[b]..cu_q[b+1];
k, v, dk, dv are [T, H, d] with cu_k; lse is [H, Tq].  Loops over sequences and heads, numpy
matrix products inside; no tiling, no online softmax.  Shares no code with the CUDA path.
"""
from __future__ import annotations

import numpy as np


def selected(level, cu_k, level_mask: int):
    """Per sequence: global indices of the encoder tokens whose level bit is set."""
    level = np.asarray(level)
    out = []
    for b in range(len(cu_k) - 1):
        idx = [i for i in range(int(cu_k[b]), int(cu_k[b + 1])) if level[i] >= 0 and (level_mask >> int(level[i])) & 1]
        out.append(np.asarray(idx, np.int64))
    return out


def forward(level, cu_k, level_mask, cu_q, qd, k, v, scale=None):
    qd, k, v = (np.asarray(x, np.float64) for x in (qd, k, v))
    Tq, H, d = qd.shape
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    o = np.zeros((Tq, H, d))
    lse = np.full((H, Tq), -np.inf)
    for b, sel in enumerate(selected(level, cu_k, level_mask)):
        r0, r1 = int(cu_q[b]), int(cu_q[b + 1])
        if len(sel) == 0 or r1 == r0:
            continue
        for h in range(H):
            a = (qd[r0:r1, h] @ k[sel, h].T) * scale
            m = a.max(axis=1, keepdims=True)
            e = np.exp(a - m)
            l = e.sum(axis=1, keepdims=True)
            o[r0:r1, h] = (e / l) @ v[sel, h]
            lse[h, r0:r1] = (m + np.log(l))[:, 0]
    return o, lse


def backward(level, cu_k, level_mask, cu_q, qd, k, v, do, scale=None):
    qd, k, v, do = (np.asarray(x, np.float64) for x in (qd, k, v, do))
    Tq, H, d = qd.shape
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    dq = np.zeros_like(qd)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    for b, sel in enumerate(selected(level, cu_k, level_mask)):
        r0, r1 = int(cu_q[b]), int(cu_q[b + 1])
        if len(sel) == 0 or r1 == r0:
            continue
        for h in range(H):
            a = (qd[r0:r1, h] @ k[sel, h].T) * scale
            e = np.exp(a - a.max(axis=1, keepdims=True))
            S = e / e.sum(axis=1, keepdims=True)
            dP = do[r0:r1, h] @ v[sel, h].T
            dS = S * (dP - (S * dP).sum(axis=1, keepdims=True))
            dv[sel, h] = S.T @ do[r0:r1, h]
            dq[r0:r1, h] = scale * dS @ k[sel, h]
            dk[sel, h] = scale * dS.T @ qd[r0:r1, h]
    return dq, dk, dv

"""Seeded synthetic inputs for the HDT hierarchical-attention path.

This module is the only code shared by the CPU oracle's tests and the CUDA
path's tests / benchmark.  It holds no arithmetic of the method itself: it
draws document hierarchies (nested lists of sentence lengths), lays them out
in document order with anchor tokens, and draws Q/K/V/dO samples.

Layout (paper, "Hierarchical Document Transformer" section and the model
hierarchy figure): a [DOC] anchor opens the document, a [SEC] anchor opens each
section, a [SENT] anchor opens each sentence, regular tokens follow their
[SENT] anchor.  Tokens stay in document order.

Structure arrays handed to both sides:
  level[i]  int8   0 [DOC], 1 [SEC], 2 [SENT], 3 regular token (deeper levels
                   allowed for generic trees), -1 PAD
  parent[i] int32  index of the parent token relative to the start of the
                   token's own sequence; -1 for the root and for PAD
  cu_seqlens int32[B+1]  cumulative sequence offsets into the packed token axis

Workloads: the paper measured on real documents (arXiv / patents / Wikipedia)
that are not available offline; the five configurations below are seeded
synthetic stand-ins with the shapes the paper's efficiency protocol states
(batch 4, 12 heads of dimension 64, lengths up to 16k / 32k tokens).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence, Tuple

import numpy as np

PAD_LEVEL = -1

Doc = List[List[int]]  # sections -> sentence lengths (regular tokens per sentence)


# ----------------------------------------------------------------------------
# layout of one document
# ----------------------------------------------------------------------------
def layout(sections: Doc) -> Tuple[np.ndarray, np.ndarray]:
    """Document-order token layout of a 3-level document.

    Returns (level int8[n], parent int32[n]) with sequence-relative parents.
    """
    level: List[int] = [0]
    parent: List[int] = [-1]
    for sec in sections:
        s = len(level)
        level.append(1)
        parent.append(0)
        for k in sec:
            t = len(level)
            level.append(2)
            parent.append(s)
            level.extend([3] * int(k))
            parent.extend([t] * int(k))
    return np.asarray(level, np.int8), np.asarray(parent, np.int32)


def layout_tree(children: Sequence) -> Tuple[np.ndarray, np.ndarray]:
    """Pre-order layout of a generic tree given as nested lists.

    `children` is the list of the root's children; every child is itself a list
    of children (an empty list is a leaf).  level = depth, root at level 0.
    """
    level: List[int] = [0]
    parent: List[int] = [-1]

    def walk(node, par, depth):
        for ch in node:
            me = len(level)
            level.append(depth)
            parent.append(par)
            walk(ch, me, depth + 1)

    walk(children, 0, 1)
    return np.asarray(level, np.int8), np.asarray(parent, np.int32)


def fit(level: np.ndarray, parent: np.ndarray, length: int, pad: bool):
    """Cut a laid-out document at `length`; optionally pad with PAD tokens."""
    n = len(level)
    if n > length:
        level, parent = level[:length], parent[:length]
    elif n < length and pad:
        extra = length - n
        level = np.concatenate([level, np.full(extra, PAD_LEVEL, np.int8)])
        parent = np.concatenate([parent, np.full(extra, -1, np.int32)])
    return level, parent


def doc_tokens(sections: Doc) -> int:
    return 1 + sum(1 + sum(1 + int(k) for k in sec) for sec in sections)


# ----------------------------------------------------------------------------
# random documents
# ----------------------------------------------------------------------------
def _u(rng, lo_hi):
    lo, hi = lo_hi
    return int(rng.integers(lo, hi + 1))


def draw_section(rng, M, K) -> List[int]:
    m = _u(rng, M)
    return [_u(rng, K) for _ in range(m)]


def gen_pad(rng, L, S, M, K):
    """n ~ U{S} sections, cut at L or padded with PAD up to L."""
    n = _u(rng, S)
    doc = [draw_section(rng, M, K) for _ in range(n)]
    lv, pa = layout(doc)
    return fit(lv, pa, L, pad=True) + (doc,)


def gen_fill(rng, L, S, M, K):
    """As gen_pad, then sections are appended until the document reaches L; cut at L."""
    n = _u(rng, S)
    doc = [draw_section(rng, M, K) for _ in range(n)]
    while doc_tokens(doc) < L:
        doc.append(draw_section(rng, M, K))
    lv, pa = layout(doc)
    return fit(lv, pa, L, pad=False) + (doc,)


def gen_pseudo(rng, L, K, per_section=32):
    """Flat text: sentences of U{K} tokens are drawn until the document reaches L and grouped into
    pseudo-sections of exactly `per_section` consecutive sentences (the last one may be shorter);
    cut at L."""
    sents = []
    total = 1
    while total < L:
        if len(sents) % per_section == 0:
            total += 1                      # the [SEC] anchor of a new pseudo-section
        k = _u(rng, K)
        sents.append(k)
        total += 1 + k
    doc = [sents[i:i + per_section] for i in range(0, len(sents), per_section)]
    lv, pa = layout(doc)
    return fit(lv, pa, L, pad=False) + (doc,)


def zipf_len(rng, a=1.5, cap=1024, clip=False) -> int:
    k = int(rng.zipf(a))
    if clip:
        return min(k, cap)
    while k > cap:
        k = int(rng.zipf(a))
    return k


def gen_skew(rng, L, frac=0.6, n_small=200, cap=1024, clip=False):
    """One section holding floor(frac*L) tokens plus n_small sections of 1-3 sentences."""
    target = int(np.floor(frac * L))
    big: List[int] = []
    used = 1  # the [SEC] anchor
    while used < target:
        k = zipf_len(rng, cap=cap, clip=clip)
        if used + 1 + k > target:
            k = target - used - 1
        big.append(k)
        used += 1 + k
    small = [[zipf_len(rng, cap=cap, clip=clip) for _ in range(_u(rng, (1, 3)))]
             for _ in range(n_small)]
    pos = _u(rng, (0, n_small))
    doc = small[:pos] + [big] + small[pos:]
    lv, pa = layout(doc)
    return fit(lv, pa, L, pad=True) + (doc,)


def random_tree(rng, max_depth: int, max_children: int, p_leaf: float = 0.3):
    """Nested-list tree of bounded depth for generic-hierarchy tests."""
    def node(depth):
        if depth >= max_depth or (depth > 0 and rng.random() < p_leaf):
            return []
        return [node(depth + 1) for _ in range(int(rng.integers(1, max_children + 1)))]
    t = node(0)
    return t


def listops_tree(rng, max_depth: int = 20, max_args: int = 5, max_len: int = 512, p_nest: float = 0.25):
    """Nested-list expression tree shaped like a ListOps sample: every operator has 2..max_args
    operands, an operand is a number (leaf) or, with probability p_nest and while depth and length
    allow, another operator; at most max_depth operator levels and max_len tokens.  The root of
    the list is the outermost operator."""
    budget = [max_len - 1]

    def op(depth):
        n_args = int(rng.integers(2, max_args + 1))
        kids = []
        for _ in range(n_args):
            if budget[0] <= 0:
                break
            budget[0] -= 1
            if depth + 1 < max_depth and budget[0] >= 3 and rng.random() < p_nest:
                kids.append(op(depth + 1))
            else:
                kids.append([])
        return kids
    return op(0)


# ----------------------------------------------------------------------------
# batches
# ----------------------------------------------------------------------------
@dataclass
class Batch:
    level: np.ndarray        # int8  [T]
    parent: np.ndarray       # int32 [T]
    cu_seqlens: np.ndarray   # int32 [B+1]
    docs: list = field(default_factory=list)  # nested lists, one per sequence (tests only)

    @property
    def total_tokens(self) -> int:
        return int(self.cu_seqlens[-1])

    @property
    def batch(self) -> int:
        return len(self.cu_seqlens) - 1

    @property
    def max_seqlen(self) -> int:
        return int(np.diff(self.cu_seqlens).max()) if self.batch else 0

    @property
    def real_tokens(self) -> int:
        return int((self.level >= 0).sum())


def pack(seqs) -> Batch:
    """Pack [(level, parent, doc?), ...] into one varlen batch."""
    lv = [np.asarray(s[0], np.int8) for s in seqs]
    pa = [np.asarray(s[1], np.int32) for s in seqs]
    cu = np.zeros(len(seqs) + 1, np.int32)
    cu[1:] = np.cumsum([len(x) for x in lv])
    docs = [s[2] if len(s) > 2 else None for s in seqs]
    if lv:
        return Batch(np.concatenate(lv), np.concatenate(pa), cu, docs)
    return Batch(np.zeros(0, np.int8), np.zeros(0, np.int32), cu, docs)


@dataclass(frozen=True)
class Config:
    name: str
    heads: int
    head_dim: int
    dtype: str          # "f32" | "bf16"
    backward: bool
    hier_seed: int
    tensor_seed: int
    description: str


CONFIGS = {
    1: Config("c1_tiny_2x3x8", 1, 64, "f32", False, 0, 0,
              "1 document, 2 sections x 3 sentences x 8 tokens (57 tokens), fp32, forward"),
    2: Config("c2_b8_L2048_pad", 12, 64, "bf16", False, 1002, 2002,
              "8 documents cut/padded to 2048; sections U{2..8}, sentences U{2..12}, tokens U{5..40}"),
    3: Config("c3_b4_L8192", 12, 64, "bf16", True, 1003, 2003,
              "4 documents of 8192 tokens; sections U{4..24}, sentences U{3..20}, tokens U{5..60}"),
    4: Config("c4_varlen16_d128", 16, 128, "bf16", True, 1004, 2004,
              "16 packed documents, lengths U{512..16384}, same generator as c3, head_dim 128"),
    5: Config("c5_skew_2x32768", 12, 64, "bf16", True, 1005, 2005,
              "2 documents of 32768: one section with 60% of tokens, Zipf(1.5) sentences capped 1024, 200 small sections"),
    # not one of the five headline configurations: flat text cut into pseudo-sections of 32 sentences
    # (the paper's setting for inputs without document structure), shape of config 3 otherwise
    6: Config("c6_pseudo32_b4_L8192", 12, 64, "bf16", True, 1006, 2006,
              "4 flat documents of 8192 tokens; pseudo-sections of 32 sentences, tokens U{5..60}"),
    # ListOps-shaped expression trees (depth <= 20, 2..5 operands, <= 512 tokens), batch 200,
    # feature dimension 128 as 2 heads x 64; used with the directed mask variants
    7: Config("c7_listops_b200_d20", 2, 64, "bf16", True, 1007, 2007,
              "200 expression trees: operators with 2..5 operands, nesting probability 0.45, depth <= 20, <= 512 tokens"),
}


def make_hierarchy(c: int, clip: bool = False) -> Batch:
    cfg = CONFIGS[c]
    rng = np.random.default_rng(cfg.hier_seed)
    if c == 1:
        doc = [[8, 8, 8], [8, 8, 8]]
        lv, pa = layout(doc)
        return pack([(lv, pa, doc)])
    if c == 2:
        return pack([gen_pad(rng, 2048, (2, 8), (2, 12), (5, 40)) for _ in range(8)])
    if c == 3:
        return pack([gen_fill(rng, 8192, (4, 24), (3, 20), (5, 60)) for _ in range(4)])
    if c == 4:
        lens = [_u(rng, (512, 16384)) for _ in range(16)]
        return pack([gen_fill(rng, L, (4, 24), (3, 20), (5, 60)) for L in lens])
    if c == 5:
        return pack([gen_skew(rng, 32768, clip=clip) for _ in range(2)])
    if c == 6:
        return pack([gen_pseudo(rng, 8192, (5, 60)) for _ in range(4)])
    if c == 7:
        return pack([layout_tree(listops_tree(rng, 20, 5, 512, 0.45)) for _ in range(200)])
    raise KeyError(c)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result stays in an fp32 container."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already bf16-representable."""
    return (np.ascontiguousarray(x, np.float32).view(np.uint32) >> 16).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32)


def make_tensors(seed: int, total_tokens: int, heads: int, head_dim: int, dtype: str,
                 names=("q", "k", "v", "do")):
    """N(0,1) samples in [T, H, d] order, one tensor after the other from one PCG64 stream.

    For dtype "bf16" the samples are rounded to bf16 and returned in fp32 containers.
    """
    rng = np.random.default_rng(seed)
    out = {}
    for nm in names:
        x = rng.standard_normal((total_tokens, heads, head_dim), dtype=np.float32)
        out[nm] = round_bf16(x) if dtype == "bf16" else x
    return out


def small_random_batch(seed: int, n_seqs=3, pad_to=None, S=(1, 4), M=(1, 4), K=(0, 9),
                       min_len=5, max_len=200) -> Batch:
    """Small random truncated / padded documents for parity and pin tests."""
    rng = np.random.default_rng(seed)
    seqs = []
    for _ in range(n_seqs):
        L = int(rng.integers(min_len, max_len + 1))
        lv, pa, doc = gen_fill(rng, L, S, M, K)
        if pad_to is not None or rng.random() < 0.3:
            tgt = pad_to if pad_to is not None else L + int(rng.integers(1, 20))
            lv, pa = fit(lv, pa, max(tgt, len(lv)), pad=True)
        seqs.append((lv, pa, doc))
    return pack(seqs)

"""Plain sequential definition of the hierarchical-attention index.  TEST INFRASTRUCTURE ONLY.

The CUDA library's ``hdt_build_index`` must reproduce every array here bit for bit.

The paper tests, tile by tile and inside its kernel, whether a tile of the mask holds a
non-zero (Algorithm 1, the "compute mask / if non-zero" steps) after sorting keys by hierarchy
level.  This build replaces that by a decomposition of the same mask that needs no sort:

*Families.*  The mask rule (parent, siblings incl. self, children) says that the pairs with
M_ij = 1 are exactly the pairs inside one *family* {q} + children(q) of some node q, for every
node q with children.  Assigning the pair (q, q) to the family of q's parent (q is its own
sibling there; the root keeps its own), every unmasked pair belongs to exactly one family.

*Stages.*  In document order (pre-order) a node whose children are all childless is directly
followed by those children, so its family is one contiguous index range.  Stage 0 handles all
such families on the full token array.  Then the children of the handled families (and PAD)
are removed; on the compacted array the next families have become contiguous, and so on until
no family is left.  Documents with [DOC]/[SEC]/[SENT] anchors need three stages: sentences on
all tokens, sections on the anchors, the document on [DOC]+[SEC].

Per stage s the index holds, for the compacted array A_s of n_s elements:
  tok[e]        global token id of element e
  par[e]        index in A_s of e's parent, -1 for a root or PAD
  rng[e]=(lo,hi) key range (indices in A_s) of row e in this stage; (0,0) when e is in no
                family handled here.  Family head q (non-root): (q+1, q+1+c); root head:
                (q, q+1+c); child of head q: (q, q+1+c), c = number of children of q.
  up[e]         index of e in A_{s+1}, -1 if removed (or no next stage)
  scu[b]        start of sequence b in A_s (cumulative, B+1 entries)
  blocks        rows (r0, r1, a, b, flags): row blocks of at most block_m (stage 0) or block_m_upper
                (stages above 0) consecutive elements of one sequence, packed greedily and cut at family boundaries when a family fits
                in a block; [a,b) = hull of the rows' key ranges (a=b=r0 if none);
                flags bit0 SELF  a>=r0 and b<=r1 (block needs no key outside itself)
                      bit1 DENSE every row's range is exactly [a,b)
                      bit2 CARRY some row has up>=0 (a partial result comes from stage s+1)
                      bit3 EMPTY no row has a key in this stage
  queue         block ids sorted by cost (r1-r0)*(b-a) descending, ties by id ascending
  queue_split   the same ids: first the n_fused blocks that are SELF and not EMPTY, then the others,
                each group in queue order
Totals: nnz = sum over stages and rows of the allowed keys in [lo, hi) (all of them under the full
rule: hi-lo; = number of unmasked pairs of the batch),
visited = sum over blocks of (r1-r0)*(b-a).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np

F_SELF, F_DENSE, F_CARRY, F_EMPTY = 1, 2, 4, 8

OK, ERR_BAD_HIERARCHY = 0, -2


@dataclass
class Stage:
    n: int
    tok: np.ndarray      # int32 [n]
    par: np.ndarray      # int32 [n]
    rng: np.ndarray      # int32 [n,2]
    up: np.ndarray       # int32 [n]
    scu: np.ndarray      # int32 [B+1]
    blocks: np.ndarray   # int32 [nb,5]
    queue: np.ndarray    # int32 [nb]
    queue_split: np.ndarray = None   # int32 [nb]: SELF non-EMPTY blocks first, each group in queue order
    n_fused: int = 0


@dataclass
class Index:
    stages: List[Stage]
    nnz: int
    visited: int


class BadHierarchy(ValueError):
    pass


def validate(level, parent, cu):
    """Preconditions on the caller's structure arrays (any violation -> BadHierarchy)."""
    B = len(cu) - 1
    if cu[0] != 0:
        raise BadHierarchy("cu_seqlens[0] != 0")
    if np.any(np.diff(cu) < 0) or int(cu[B]) != len(level):
        raise BadHierarchy("cu_seqlens not monotone or not ending at the token count")
    for b in range(B):
        s0, s1 = int(cu[b]), int(cu[b + 1])
        if s1 < s0:
            raise BadHierarchy("cu_seqlens not monotone")
        seen_pad = False
        for i in range(s0, s1):
            l, p = int(level[i]), int(parent[i])
            if l < 0:
                if l != -1 or p != -1:
                    raise BadHierarchy("PAD must have level -1 and parent -1")
                seen_pad = True
                continue
            if seen_pad:
                raise BadHierarchy("PAD only as a suffix")
            r = i - s0
            if r == 0:
                if l != 0 or p != -1:
                    raise BadHierarchy("first token must be the level-0 root")
            else:
                if not (0 <= p < r):
                    raise BadHierarchy("parent must precede the token inside its sequence")
                if int(level[s0 + p]) != l - 1:
                    raise BadHierarchy("level must be parent's level + 1")


def pair_allowed(e: int, j: int, lo: int, directions: int) -> bool:
    """Direction bits on one entry (row e, key j) of a stage whose row range starts at lo.
    A row whose range starts at or after itself is the head of its family (the keys after it are
    its children); otherwise lo is the row's parent and the other keys are its siblings.
    Bits: 1 = a token attends to its parent, 2 = to its other siblings, 4 = to its children; the
    diagonal always stays (paper, "Mathematical Reasoning Tasks": the ListOps attention patterns)."""
    if j == e:
        return True
    if lo >= e:
        return bool(directions & 4)
    return bool(directions & (1 if j == lo else 2))


def row_pairs(e: int, lo: int, hi: int, directions: int) -> int:
    """Number of allowed keys of row e with range [lo, hi)."""
    if hi <= lo:
        return 0
    if lo >= e:
        return (1 if lo == e else 0) + ((hi - e - 1) if directions & 4 else 0)
    return 1 + (1 if directions & 1 else 0) + ((hi - lo - 2) if directions & 2 else 0)


def build(level, parent, cu, block_m: int = 128, max_stages: int = 32, block_m_upper: int = 128,
          directions: int = 7) -> Index:
    level = np.asarray(level, np.int8)
    parent = np.asarray(parent, np.int32)
    cu = np.asarray(cu, np.int32)
    validate(level, parent, cu)
    B = len(cu) - 1
    T = int(cu[B])

    # stage 0 arrays
    tok = np.arange(T, dtype=np.int32)
    par = np.full(T, -1, np.int32)
    real = np.zeros(T, bool)
    for b in range(B):
        for i in range(int(cu[b]), int(cu[b + 1])):
            if level[i] >= 0:
                real[i] = True
                if parent[i] >= 0:
                    par[i] = cu[b] + parent[i]
    scu = cu.copy()

    stages: List[Stage] = []
    nnz = 0
    visited = 0
    s = 0
    while True:
        n = len(tok)
        cnt = np.zeros(n, np.int64)
        for e in range(n):
            if par[e] >= 0:
                cnt[par[e]] += 1
        nlc = np.zeros(n, np.int64)          # children that have children themselves
        for e in range(n):
            if par[e] >= 0 and cnt[e] > 0:
                nlc[par[e]] += 1
        head = np.zeros(n, bool)
        for e in range(n):
            if not real[e]:
                continue
            if cnt[e] > 0 and nlc[e] == 0:
                head[e] = True
            elif s == 0 and par[e] < 0 and cnt[e] == 0:
                head[e] = True               # a document that is only its root: the pair (root, root)
        if s > 0 and not head.any():
            break                            # nothing left to handle: previous stage was the last
        if len(stages) >= max_stages:
            raise BadHierarchy("hierarchy deeper than max_stages")

        rng = np.zeros((n, 2), np.int32)
        uid = np.full(n, -1, np.int64)       # family (head index) of each element in this stage
        for e in range(n):
            if head[e]:
                c = int(cnt[e])
                rng[e] = (e, e + 1 + c) if par[e] < 0 else (e + 1, e + 1 + c)
                uid[e] = e
        for e in range(n):
            p = par[e]
            if p >= 0 and head[p]:
                c = int(cnt[p])
                if not (p < e <= p + c):
                    raise BadHierarchy("children of a node must follow it in document order")
                rng[e] = (p, p + 1 + c)
                uid[e] = p
        nnz += sum(row_pairs(e, int(rng[e, 0]), int(rng[e, 1]), directions) for e in range(n))

        # removal for the next stage
        keep = np.zeros(n, bool)
        for e in range(n):
            keep[e] = real[e] and not (par[e] >= 0 and head[par[e]])
        new_of = np.cumsum(keep) - 1
        # does a next stage exist?  It does iff some kept element heads a family there.
        n2 = int(keep.sum())
        tok2 = tok[keep]
        par2 = np.where(par[keep] >= 0, new_of[np.maximum(par[keep], 0)], -1).astype(np.int32)
        cnt2 = np.zeros(n2, np.int64)
        for e in range(n2):
            if par2[e] >= 0:
                cnt2[par2[e]] += 1
        has_next = bool((cnt2 > 0).any())
        up = np.where(keep & has_next, new_of, -1).astype(np.int32)

        # row blocks
        blocks = []
        for b in range(B):
            pos, end_seq = int(scu[b]), int(scu[b + 1])
            bm = block_m if s == 0 else block_m_upper    # stages above 0 use their own block size
            while pos < end_seq:
                end = min(pos + bm, end_seq)
                if end < end_seq and uid[end] >= 0 and uid[end] == uid[end - 1] and uid[end] > pos:
                    end = int(uid[end])
                a, bb, any_key, dense, carry = None, None, False, True, False
                for e in range(pos, end):
                    lo, hi = int(rng[e, 0]), int(rng[e, 1])
                    if hi > lo:
                        any_key = True
                        a = lo if a is None else min(a, lo)
                        bb = hi if bb is None else max(bb, hi)
                    if up[e] >= 0:
                        carry = True
                if not any_key:
                    a = bb = pos
                for e in range(pos, end):
                    if not (rng[e, 0] == a and rng[e, 1] == bb):
                        dense = False
                fl = 0
                if a >= pos and bb <= end:
                    fl |= F_SELF
                if dense and any_key:
                    fl |= F_DENSE
                if carry:
                    fl |= F_CARRY
                if not any_key:
                    fl |= F_EMPTY
                blocks.append((pos, end, a, bb, fl))
                visited += (end - pos) * (bb - a)
                pos = end
        blocks = np.asarray(blocks, np.int32).reshape(-1, 5)
        cost = (blocks[:, 1] - blocks[:, 0]).astype(np.int64) * (blocks[:, 3] - blocks[:, 2]).astype(np.int64)
        queue = np.asarray(sorted(range(len(blocks)), key=lambda i: (-int(cost[i]), i)), np.int32)

        elig = [bool(f & F_SELF) and not (f & F_EMPTY) for f in blocks[:, 4]] if len(blocks) else []
        queue_split = np.asarray([i for i in queue if elig[i]] + [i for i in queue if not elig[i]], np.int32)
        stages.append(Stage(n, tok.copy(), par.copy(), rng, up, scu.copy(), blocks, queue, queue_split,
                            int(sum(elig))))

        if not has_next:
            break
        # compact to the next stage
        scu2 = np.zeros(B + 1, np.int32)
        for b in range(B):
            scu2[b + 1] = scu2[b] + int(keep[int(scu[b]):int(scu[b + 1])].sum())
        tok, par, scu = tok2.astype(np.int32), par2, scu2
        real = np.ones(n2, bool)
        s += 1

    return Index(stages, nnz, visited)


def pairs_of(index: Index, T: int, directions: int = 7) -> np.ndarray:
    """Count matrix [T,T] of how often each (query token, key token) pair is covered."""
    C = np.zeros((T, T), np.int32)
    for st in index.stages:
        for e in range(st.n):
            lo, hi = st.rng[e]
            for j in range(lo, hi):
                if pair_allowed(e, j, int(lo), directions):
                    C[st.tok[e], st.tok[j]] += 1
    return C

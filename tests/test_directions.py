"""Pins for the directed mask variants (paper, "Mathematical Reasoning Tasks": the ListOps attention
patterns; full rule = all three groups, "operands do not attend to their operators" = without the
child->parent group, "operands do not attend to each other" = additionally without the sibling
group).  Sources of truth other than the oracle: a walk over the generator's nested lists, set
algebra between the variants, closed forms, numpy masked attention and its textbook gradient."""
import numpy as np
import pytest

import gen
import oracle
from oracle import index_oracle as ix

UP, SIB, DOWN = 1, 2, 4


def one(level, parent):
    return np.asarray(level, np.int8), np.asarray(parent, np.int32), np.array([0, len(level)], np.int32)


def groups_from_nested_lists(tree):
    """Pre-order numbering of the nested lists (root = 0) and the three entry groups as sets of
    (row, key): a child attending its parent, siblings attending each other, a parent attending a
    child.  Written from the lists alone: no level or parent array is consulted."""
    up, sib, down = set(), set(), set()
    counter = [1]

    def walk(children, me):
        ids = []
        for ch in children:
            c = counter[0]
            counter[0] += 1
            ids.append(c)
            walk(ch, c)
        for a in ids:
            up.add((a, me))
            down.add((me, a))
            for b in ids:
                if a != b:
                    sib.add((a, b))

    walk(tree, 0)
    return counter[0], up, sib, down


def mask_from_groups(n, up, sib, down, d):
    M = np.eye(n, dtype=np.uint8)
    for bit, grp in ((UP, up), (SIB, sib), (DOWN, down)):
        if d & bit:
            for (i, j) in grp:
                M[i, j] = 1
    return M


def trees(seed, count, depth=5, kids=4):
    rng = np.random.default_rng(seed)
    return [gen.random_tree(rng, int(rng.integers(1, depth + 1)), kids) for _ in range(count)]


@pytest.mark.parametrize("d", range(8))
def test_directed_mask_equals_walk_over_nested_lists(d):
    for tree in trees(11, 25) + [gen.listops_tree(np.random.default_rng(3), 6, 5, 80, 0.5)]:
        lv, pa = gen.layout_tree(tree)
        n, up, sib, down = groups_from_nested_lists(tree)
        assert n == len(lv)
        assert np.array_equal(oracle.mask(*one(lv, pa), 0, directions=d), mask_from_groups(n, up, sib, down, d))


def test_set_algebra_between_variants():
    for tree in trees(12, 10):
        lv, pa = gen.layout_tree(tree)
        M = {d: oracle.mask(*one(lv, pa), 0, directions=d) for d in range(8)}
        n = len(lv)
        assert np.array_equal(M[7], oracle.mask(*one(lv, pa), 0))            # default = full rule
        assert np.array_equal(M[0], np.eye(n, dtype=np.uint8))               # the diagonal always stays
        assert np.array_equal(M[UP].T, M[DOWN])                              # a parent's child is that child's parent
        assert np.array_equal(M[SIB], M[SIB].T)
        assert np.array_equal(M[7], M[UP] | M[SIB] | M[DOWN])
        for d in range(8):
            assert np.array_equal(M[d], M[d & UP] | M[d & SIB] | M[d & DOWN])
        # counts: one parent entry per non-root node in each direction
        assert M[UP].sum() == n + (n - 1) and M[DOWN].sum() == n + (n - 1)


def test_config1_direction_counts():
    b = gen.make_hierarchy(1)      # 57 tokens: 56 parent links, 350 ordered sibling pairs
    got = {d: int(oracle.mask(b.level, b.parent, b.cu_seqlens, 0, directions=d).sum()) for d in (0, UP, SIB, DOWN, 6, 7)}
    assert got == {0: 57, UP: 113, SIB: 407, DOWN: 113, 6: 463, 7: 519}


def test_padding_stays_out():
    lv, pa = gen.layout([[2, 1], [3]])
    lv, pa = gen.fit(lv, pa, len(lv) + 4, pad=True)
    for d in range(8):
        M = oracle.mask(*one(lv, pa), 0, directions=d)
        assert M[-4:].sum() == 0 and M[:, -4:].sum() == 0


def dense(q, k, v, mask, scale):
    a = np.where(mask.astype(bool), (q @ k.T) * scale, -np.inf)
    m = a.max(1, keepdims=True)
    e = np.exp(a - m)
    S = e / e.sum(1, keepdims=True)
    return S @ v, (m + np.log(e.sum(1, keepdims=True)))[:, 0], S


@pytest.mark.parametrize("d", [6, 4, 5, 3])
def test_forward_and_backward_equal_numpy_masked_attention(d):
    tree = gen.listops_tree(np.random.default_rng(8), 5, 4, 60, 0.5)
    lv, pa = gen.layout_tree(tree)
    n, up, sib, down = groups_from_nested_lists(tree)
    M = mask_from_groups(n, up, sib, down, d)
    rng = np.random.default_rng(9)
    H, dim = 2, 8
    q, k, v, do = (rng.standard_normal((n, H, dim)) for _ in range(4))
    o, lse = oracle.forward(*one(lv, pa), q, k, v, directions=d)
    dq, dk, dv = oracle.backward(*one(lv, pa), q, k, v, do, directions=d)
    sc = 1 / np.sqrt(dim)
    for h in range(H):
        o_n, lse_n, S = dense(q[:, h], k[:, h], v[:, h], M, sc)
        assert np.allclose(o[:, h], o_n, atol=1e-13) and np.allclose(lse[h], lse_n, atol=1e-13)
        dP = do[:, h] @ v[:, h].T
        dS = S * (dP - (S * dP).sum(1, keepdims=True))
        assert np.allclose(dv[:, h], S.T @ do[:, h], atol=1e-13)
        assert np.allclose(dq[:, h], sc * dS @ k[:, h], atol=1e-13)
        assert np.allclose(dk[:, h], sc * dS.T @ q[:, h], atol=1e-13)
    # sampled rows / keys agree with the full functions under the same bits
    rows = np.arange(0, n, 3, dtype=np.int32)
    o_r, lse_r, dq_r = oracle.rows(*one(lv, pa), q, k, v, rows, do=do, directions=d)
    dk_c, dv_c = oracle.cols(*one(lv, pa), q, k, v, do, rows, directions=d)
    assert np.allclose(o_r, o[rows]) and np.allclose(lse_r, lse[:, rows].T) and np.allclose(dq_r, dq[rows])
    assert np.allclose(dk_c, dk[rows]) and np.allclose(dv_c, dv[rows])


def test_parent_to_child_only_closed_forms():
    """Only parent -> child entries kept: a leaf attends to itself alone, so O = V, LSE = q.k scale,
    and no gradient reaches it as a query (dQ = 0)."""
    tree = gen.listops_tree(np.random.default_rng(2), 4, 5, 40, 0.4)
    lv, pa = gen.layout_tree(tree)
    n = len(lv)
    leaf = np.ones(n, bool)
    leaf[pa[pa >= 0]] = False
    rng = np.random.default_rng(4)
    q, k, v, do = (rng.standard_normal((n, 1, 8)) for _ in range(4))
    o, lse = oracle.forward(*one(lv, pa), q, k, v, directions=DOWN)
    dq, dk, dv = oracle.backward(*one(lv, pa), q, k, v, do, directions=DOWN)
    assert np.allclose(o[leaf], v[leaf], atol=1e-14)
    assert np.allclose(lse[0, leaf], (q[leaf, 0] * k[leaf, 0]).sum(-1) / np.sqrt(8), atol=1e-14)
    assert np.abs(dq[leaf]).max() < 1e-14


# ----------------------------------------------------------------------------------------
# index: the staged ranges, filtered by the bits, cover exactly the directed mask
# ----------------------------------------------------------------------------------------
@pytest.mark.parametrize("d", range(8))
def test_index_pairs_cover_directed_mask_exactly_once(d):
    rng = np.random.default_rng(20 + d)
    seqs = [gen.layout_tree(t) for t in trees(30 + d, 4, depth=6)] + [gen.gen_fill(rng, 70, (1, 3), (1, 3), (0, 6))[:2]]
    b = gen.pack(seqs)
    idx = ix.build(b.level, b.parent, b.cu_seqlens, 16, block_m_upper=8, directions=d)
    C = ix.pairs_of(idx, b.total_tokens, d)
    M = np.zeros_like(C)
    for s in range(b.batch):
        a, z = b.cu_seqlens[s], b.cu_seqlens[s + 1]
        M[a:z, a:z] = oracle.mask(b.level, b.parent, b.cu_seqlens, s, directions=d)
    assert np.array_equal(C, M)
    assert idx.nnz == int(M.sum())
    # the ranges themselves do not depend on the bits
    full = ix.build(b.level, b.parent, b.cu_seqlens, 16, block_m_upper=8)
    for sa, sb in zip(idx.stages, full.stages):
        assert np.array_equal(sa.rng, sb.rng) and np.array_equal(sa.blocks, sb.blocks)

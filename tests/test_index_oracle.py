"""Pins for the index definition: the staged family decomposition must cover exactly the
unmasked pairs of the dense mask (brute force), each once, on documents and generic trees."""
import numpy as np
import pytest

import gen
import oracle
from oracle import index_oracle as ix


def dense_batch_mask(b):
    T = b.total_tokens
    M = np.zeros((T, T), np.int32)
    for s in range(b.batch):
        lo, hi = b.cu_seqlens[s], b.cu_seqlens[s + 1]
        M[lo:hi, lo:hi] = oracle.mask(b.level, b.parent, b.cu_seqlens, s)
    return M


def check_structure(b, idx, block_m):
    T = b.total_tokens
    M = dense_batch_mask(b)
    assert np.array_equal(ix.pairs_of(idx, T), M)          # every unmasked pair exactly once
    assert idx.nnz == M.sum()
    vis = 0
    for si, st in enumerate(idx.stages):
        # blocks tile every sequence of the stage array, never straddle, never exceed block_m
        pos = 0
        for r0, r1, a, bb, fl in st.blocks:
            assert r0 == pos and r0 < r1 <= r0 + block_m
            seq = np.searchsorted(st.scu, r0, side="right") - 1
            assert r1 <= st.scu[seq + 1]
            rows = st.rng[r0:r1]
            live = rows[:, 1] > rows[:, 0]
            if live.any():
                assert a == rows[live, 0].min() and bb == rows[live, 1].max()
                assert st.scu[seq] <= a and bb <= st.scu[seq + 1]
            else:
                assert a == bb == r0
            assert bool(fl & ix.F_EMPTY) == (not live.any())
            assert bool(fl & ix.F_SELF) == (a >= r0 and bb <= r1)
            assert bool(fl & ix.F_DENSE) == (live.all() and (rows[:, 0] == a).all() and (rows[:, 1] == bb).all())
            assert bool(fl & ix.F_CARRY) == bool((st.up[r0:r1] >= 0).any())
            vis += (r1 - r0) * (bb - a)
            pos = r1
        assert pos == st.n == st.scu[-1]
        cost = (st.blocks[:, 1] - st.blocks[:, 0]).astype(np.int64) * (st.blocks[:, 3] - st.blocks[:, 2])
        q = st.queue
        assert sorted(q.tolist()) == list(range(len(st.blocks)))
        for x, y in zip(q[:-1], q[1:]):
            assert (cost[x], -x) >= (cost[y], -y)
        elig = [(f & ix.F_SELF) and not (f & ix.F_EMPTY) for f in st.blocks[:, 4]]
        assert st.n_fused == sum(bool(x) for x in elig)
        assert all(elig[i] for i in st.queue_split[:st.n_fused])
        assert not any(elig[i] for i in st.queue_split[st.n_fused:])
        assert sorted(st.queue_split.tolist()) == list(range(len(st.blocks)))
        # up / tok maps
        if si + 1 < len(idx.stages):
            nx = idx.stages[si + 1]
            kept = np.flatnonzero(st.up >= 0)
            assert np.array_equal(st.up[kept], np.arange(nx.n))
            assert np.array_equal(st.tok[kept], nx.tok)
        else:
            assert (st.up == -1).all()
    assert vis == idx.visited


@pytest.mark.parametrize("block_m", [128, 16, 5])
def test_documents(block_m):
    for seed in range(12):
        b = gen.small_random_batch(seed, n_seqs=3, max_len=160)
        idx = ix.build(b.level, b.parent, b.cu_seqlens, block_m, block_m_upper=block_m)
        check_structure(b, idx, block_m)
        assert len(idx.stages) <= 3
        idx = ix.build(b.level, b.parent, b.cu_seqlens, 128, block_m_upper=block_m)
        check_structure(b, idx, 128)


def test_three_stages_on_config1_and_family_alignment():
    b = gen.make_hierarchy(1)
    idx = ix.build(b.level, b.parent, b.cu_seqlens, 128)
    check_structure(b, idx, 128)
    assert [st.n for st in idx.stages] == [57, 9, 3]
    assert idx.nnz == 519
    # stage 0: 6 sentence families of 9; each head sees its 8 tokens, each token all 9
    st = idx.stages[0]
    assert (st.rng[:, 1] - st.rng[:, 0]).tolist().count(9) == 48
    assert (st.rng[:, 1] - st.rng[:, 0]).tolist().count(8) == 6
    # with block_m = 20 blocks are cut at sentence boundaries: 2 sentences (18 rows) per block
    idx = ix.build(b.level, b.parent, b.cu_seqlens, 20)
    for r0, r1, a, bb, fl in idx.stages[0].blocks:
        if not fl & ix.F_EMPTY:
            assert fl & ix.F_SELF


def test_generic_trees_and_degenerate_documents():
    rng = np.random.default_rng(2)
    seqs = []
    for t in range(30):
        tree = gen.random_tree(rng, max_depth=int(rng.integers(1, 7)), max_children=5)
        seqs.append(gen.layout_tree(tree))
    seqs.append((np.array([0], np.int8), np.array([-1], np.int32)))                 # root only
    seqs.append((np.array([0, -1, -1], np.int8), np.array([-1, -1, -1], np.int32)))  # root + PAD
    seqs.append((np.array([-1, -1], np.int8), np.array([-1, -1], np.int32)))        # PAD only
    seqs.append((np.zeros(0, np.int8), np.zeros(0, np.int32)))                      # empty sequence
    seqs.append(gen.layout([[300, 2], [1]]))                                        # family longer than a block
    b = gen.pack(seqs)
    for bm in (128, 7):
        idx = ix.build(b.level, b.parent, b.cu_seqlens, bm, block_m_upper=bm)
        check_structure(b, idx, bm)


def test_long_family_is_split_and_dense():
    lv, pa = gen.layout([[300]])
    b = gen.pack([(lv, pa)])
    idx = ix.build(b.level, b.parent, b.cu_seqlens, 128)
    st = idx.stages[0]
    # the sentence (head at 2, 300 tokens) does not fit: the cut backs off to its start, then
    # it is split into pieces of block_m rows
    assert st.blocks[:, :2].tolist() == [[0, 2], [2, 130], [130, 258], [258, 303]]
    assert st.blocks[1, 2] == 2 and st.blocks[1, 3] == 303 and not st.blocks[1, 4] & ix.F_DENSE
    assert st.blocks[2, 2] == 2 and st.blocks[2, 3] == 303 and st.blocks[2, 4] & ix.F_DENSE
    assert not st.blocks[2, 4] & ix.F_SELF


def test_bad_hierarchies_are_rejected():
    lv, pa = gen.layout([[2, 1], [1]])
    cu = np.array([0, 10], np.int32)
    bad = pa.copy(); bad[3] = 5                    # parent after the token
    with pytest.raises(ix.BadHierarchy):
        ix.build(lv, bad, cu)
    bad = pa.copy(); bad[6] = 2                    # right level, but not in document order
    with pytest.raises(ix.BadHierarchy):
        ix.build(lv, bad, cu)
    badl = lv.copy(); badl[3] = 2                  # level jump
    with pytest.raises(ix.BadHierarchy):
        ix.build(badl, pa, cu)
    badl = lv.copy(); badl[0] = 1                  # no root
    with pytest.raises(ix.BadHierarchy):
        ix.build(badl, pa, cu)
    lvp = np.concatenate([lv[:4], [-1], lv[5:]]).astype(np.int8)   # PAD in the middle
    pap = pa.copy(); pap[4] = -1
    with pytest.raises(ix.BadHierarchy):
        ix.build(lvp, pap, cu)
    with pytest.raises(ix.BadHierarchy):
        ix.build(lv, pa, np.array([0, 12, 10], np.int32))

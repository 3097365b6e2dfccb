"""Pins for the CPU oracle: each test ties a part of it to something other than itself.

Sources of truth used here: the paper's rule in words (parent / siblings / children), its
per-level mask equations on hierarchy index vectors, a hand-worked 10-token document, closed
forms, reductions to dense softmax attention written with numpy library calls, central finite
differences, and brute-force tree walks over the generator's nested lists.
"""
import os

import numpy as np
import pytest

import gen
import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------------------
# independent derivations of the mask
# ----------------------------------------------------------------------------------------
def pvectors(level):
    """Hierarchy index vectors p=(p1,p2,p3): section number, sentence number in its section,
    token number in its sentence; an anchor carries 0 on every level below its own."""
    n = len(level)
    p = np.zeros((n, 3), int)
    sec = sent = tok = 0
    for i in range(n):
        l = level[i]
        if l == 0:
            sec = sent = tok = 0
        elif l == 1:
            sec += 1; sent = 0; tok = 0
        elif l == 2:
            sent += 1; tok = 0
        elif l == 3:
            tok += 1
        p[i] = (sec, sent, tok)
    return p


def mask_from_equations(p):
    """OR of the DOC / SEC / SENT masks of the paper's attention-mask equations."""
    p1, p2, p3 = p[:, 0], p[:, 1], p[:, 2]
    m_doc = (p2[:, None] == 0) & (p2[None, :] == 0)
    m_sec = (p3[:, None] == 0) & (p3[None, :] == 0) & (p1[:, None] == p1[None, :])
    m_sent = (p1[:, None] == p1[None, :]) & (p2[:, None] == p2[None, :])
    return (m_doc | m_sec | m_sent).astype(np.uint8)


def mask_from_tree_walk(doc, n):
    """Enumerate, per node of the nested lists, the node with its children: all pairs inside
    such a family attend to each other (a family = one box of the hierarchy figure)."""
    M = np.zeros((n, n), np.uint8)
    pos = 1
    fam_doc = [0]
    families = []
    for sec in doc:
        s = pos; pos += 1
        fam_doc.append(s)
        fam_sec = [s]
        for k in sec:
            t = pos; pos += 1
            fam_sec.append(t)
            fam_sent = [t] + list(range(pos, pos + k))
            pos += k
            families.append(fam_sent)
        families.append(fam_sec)
    families.append(fam_doc)
    for fam in families:
        fam = [x for x in fam if x < n]          # truncation cuts the token list
        for a in fam:
            for b in fam:
                M[a, b] = 1
    return M


def one(level, parent):
    return np.asarray(level, np.int8), np.asarray(parent, np.int32), np.array([0, len(level)], np.int32)


def test_hand_worked_mask():
    rows = [l.split() for l in open(os.path.join(GOLD, "hand_mask_10tok.txt")) if not l.startswith("#")]
    level = [int(r[2]) for r in rows]
    parent = [int(r[3]) for r in rows]
    want = np.array([[c == "1" for c in r[4]] for r in rows], np.uint8)
    lv, pa = gen.layout([[2, 1], [1]])
    assert lv.tolist() == level and pa.tolist() == parent
    got = oracle.mask(*one(level, parent), 0)
    assert np.array_equal(got, want)
    assert got.sum() == 34
    assert got.sum(1).tolist() == [3, 5, 5, 3, 3, 4, 2, 4, 3, 2]


def test_three_derivations_agree():
    rng = np.random.default_rng(7)
    for t in range(150):
        L = int(rng.integers(1, 300))
        lv, pa, doc = gen.gen_fill(rng, L, (1, 4), (1, 4), (0, 9))
        M = oracle.mask(*one(lv, pa), 0)
        assert np.array_equal(M, mask_from_equations(pvectors(lv))), t
        assert np.array_equal(M, mask_from_tree_walk(doc, L)), t


def test_config1_counts():
    b = gen.make_hierarchy(1)
    assert b.total_tokens == 57
    M = oracle.mask(b.level, b.parent, b.cu_seqlens, 0)
    assert M.sum() == 519
    deg, cnt = np.unique(M.sum(1), return_counts=True)
    # [DOC] 1+2, [SEC] 1+2+3, [SENT] 1+3+8, regular token 1+8
    assert dict(zip(deg.tolist(), cnt.tolist())) == {3: 1, 6: 2, 12: 6, 9: 48}


def test_nnz_closed_form_and_degrees():
    rng = np.random.default_rng(11)
    for t in range(100):
        L = int(rng.integers(1, 400))
        lv, pa, _ = gen.gen_fill(rng, L, (1, 5), (1, 5), (0, 12))
        M = oracle.mask(*one(lv, pa), 0)
        ch = np.bincount(pa[pa >= 0], minlength=L)
        # deg(i) = [has parent] + #siblings incl. self + #children
        sib = np.where(pa >= 0, ch[np.maximum(pa, 0)], 1)
        deg = (pa >= 0).astype(int) + sib + ch
        assert np.array_equal(M.sum(1), deg)
        heads = np.flatnonzero(ch > 0)
        nnz = int(((1 + ch[heads]) ** 2).sum()) - int((heads != 0).sum()) if L > 1 else 1
        assert nnz == M.sum()


def test_mask_invariants_and_padding():
    b = gen.small_random_batch(3, n_seqs=4, pad_to=150, max_len=140)
    for s in range(b.batch):
        lo, hi = b.cu_seqlens[s], b.cu_seqlens[s + 1]
        lv, pa = b.level[lo:hi], b.parent[lo:hi]
        M = oracle.mask(b.level, b.parent, b.cu_seqlens, s)
        assert np.array_equal(M, M.T)
        real = lv >= 0
        assert (M.diagonal() == real).all()
        assert M[~real].sum() == 0 and M[:, ~real].sum() == 0
        n = hi - lo
        # tree distance: pairs at distance <= 1, or 2 through a common parent; never grandparent
        for i in range(n):
            if not real[i] or pa[i] < 0 or pa[pa[i]] < 0:
                continue
            g = pa[pa[i]]
            assert M[i, g] == 0 and M[g, i] == 0
    # regular tokens of different sentences are not connected (model-hierarchy figure: T1, T3)
    lv, pa = gen.layout([[2, 2]])
    M = oracle.mask(*one(lv, pa), 0)
    t1, t3 = 3, 6
    assert lv[t1] == 3 and lv[t3] == 3 and pa[t1] != pa[t3]
    assert M[t1, t3] == 0


def test_generic_depth_trees_tree_distance():
    rng = np.random.default_rng(5)
    for t in range(40):
        tree = gen.random_tree(rng, max_depth=int(rng.integers(1, 6)), max_children=4)
        lv, pa = gen.layout_tree(tree)
        n = len(lv)
        M = oracle.mask(*one(lv, pa), 0)
        for i in range(n):
            for j in range(n):
                want = (i == j) or pa[i] == j or pa[j] == i or (pa[i] >= 0 and pa[i] == pa[j])
                assert M[i, j] == int(want)


# ----------------------------------------------------------------------------------------
# forward
# ----------------------------------------------------------------------------------------
def dense_attention_numpy(q, k, v, mask, scale):
    """Textbook masked softmax attention for one head with numpy library calls."""
    a = (q @ k.T) * scale
    a = np.where(mask.astype(bool), a, -np.inf)
    m = a.max(1, keepdims=True)
    e = np.exp(a - m)
    l = e.sum(1, keepdims=True)
    return (e / l) @ v, (m + np.log(l))[:, 0], e / l


def rand_qkv(seed, T, H, d, names=("q", "k", "v", "do")):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((T, H, d)) for _ in names]


def test_probabilities_rows_sum_to_one_and_zero_where_masked():
    b = gen.small_random_batch(21, n_seqs=2, max_len=120)
    q, k, v, _ = rand_qkv(1, b.total_tokens, 2, 8)
    for s in range(b.batch):
        M = oracle.mask(b.level, b.parent, b.cu_seqlens, s)
        S = oracle.probs(b.level, b.parent, b.cu_seqlens, q, k, s, 1)
        real = b.level[b.cu_seqlens[s]:b.cu_seqlens[s + 1]] >= 0
        assert np.all(S[M == 0] == 0.0)
        assert np.allclose(S[real].sum(1), 1.0, atol=1e-14)
        assert np.all(S[~real] == 0.0)


def test_zero_queries_give_uniform_attention():
    b = gen.small_random_batch(22, n_seqs=2, max_len=90)
    q, k, v, _ = rand_qkv(2, b.total_tokens, 2, 8)
    q[:] = 0.0
    o, lse = oracle.forward(b.level, b.parent, b.cu_seqlens, q, k, v)
    for s in range(b.batch):
        lo, hi = b.cu_seqlens[s], b.cu_seqlens[s + 1]
        M = oracle.mask(b.level, b.parent, b.cu_seqlens, s).astype(float)
        deg = M.sum(1)
        for h in range(2):
            want = np.where(deg[:, None] > 0, (M @ v[lo:hi, h]) / np.maximum(deg, 1)[:, None], 0.0)
            assert np.allclose(o[lo:hi, h], want, atol=1e-13)
            with np.errstate(divide="ignore"):
                assert np.allclose(lse[h, lo:hi], np.log(deg), atol=1e-13)


def test_mask_readout_config1():
    """Q = 0 and V = leading columns of the identity give O_ij = M_ij / deg(i)."""
    b = gen.make_hierarchy(1)
    T, d = b.total_tokens, 64
    q = np.zeros((T, 1, d)); k = np.random.default_rng(3).standard_normal((T, 1, d))
    v = np.zeros((T, 1, d)); v[np.arange(T), 0, np.arange(T)] = 1.0
    o, _ = oracle.forward(b.level, b.parent, b.cu_seqlens, q, k, v)
    M = mask_from_tree_walk(b.docs[0], T).astype(float)
    assert np.allclose(o[:, 0, :T], M / M.sum(1, keepdims=True), atol=1e-15)
    assert np.all(o[:, 0, T:] == 0)


def test_reduces_to_dense_attention():
    # (ii) a one-family hierarchy (root whose children are all other tokens): every row is dense
    n, H, d = 23, 2, 8
    lv = np.array([0] + [1] * (n - 1), np.int8); pa = np.array([-1] + [0] * (n - 1), np.int32)
    q, k, v, _ = rand_qkv(4, n, H, d)
    o, lse = oracle.forward(*one(lv, pa), q, k, v)
    for h in range(H):
        od, ld, _ = dense_attention_numpy(q[:, h], k[:, h], v[:, h], np.ones((n, n)), 1 / np.sqrt(d))
        assert np.allclose(o[:, h], od, atol=1e-13) and np.allclose(lse[h], ld, atol=1e-13)
    # (i) single section, single sentence: regular-token rows = dense attention over {SENT} + tokens
    lv, pa = gen.layout([[9]])
    n = len(lv)
    q, k, v, _ = rand_qkv(5, n, H, d)
    o, lse = oracle.forward(*one(lv, pa), q, k, v)
    keys = np.arange(2, n)      # [SENT] at 2, its tokens after it
    for h in range(H):
        od, ld, _ = dense_attention_numpy(q[3:, h], k[keys, h], v[keys, h], np.ones((n - 3, len(keys))),
                                          1 / np.sqrt(d))
        assert np.allclose(o[3:, h], od, atol=1e-13) and np.allclose(lse[h, 3:], ld, atol=1e-13)


def test_against_numpy_masked_attention_with_tree_walk_mask():
    rng = np.random.default_rng(6)
    H, d = 3, 16
    for t in range(5):
        L = int(rng.integers(20, 160))
        lv, pa, doc = gen.gen_fill(rng, L, (1, 4), (1, 5), (0, 12))
        q, k, v, _ = rand_qkv(100 + t, L, H, d)
        o, lse = oracle.forward(*one(lv, pa), q, k, v, scale=0.37)
        M = mask_from_tree_walk(doc, L)
        for h in range(H):
            od, ld, _ = dense_attention_numpy(q[:, h], k[:, h], v[:, h], M, 0.37)
            assert np.allclose(o[:, h], od, atol=1e-12) and np.allclose(lse[h], ld, atol=1e-12)


def test_family_decomposition_lse_merge():
    """A row's output is the LSE-merge of dense attention over its parent's family and over its
    own family, with the row's own key counted once."""
    lv, pa = gen.layout([[4, 3], [5]])
    n, H, d = len(lv), 1, 8
    q, k, v, _ = rand_qkv(8, n, H, d)
    o, lse = oracle.forward(*one(lv, pa), q, k, v)
    sc = 1 / np.sqrt(d)
    for i in range(n):
        fam_up = [j for j in range(n) if pa[i] >= 0 and (j == pa[i] or pa[j] == pa[i])] or [i]
        fam_dn = [j for j in range(n) if pa[j] == i]
        parts = []
        for keys in (fam_up, fam_dn):
            if not keys:
                continue
            a = (k[keys, 0] @ q[i, 0]) * sc
            m = a.max(); e = np.exp(a - m)
            parts.append((m + np.log(e.sum()), (e / e.sum()) @ v[keys, 0]))
        L = np.logaddexp.reduce([p[0] for p in parts])
        out = sum(np.exp(p[0] - L) * p[1] for p in parts)
        assert np.allclose(o[i, 0], out, atol=1e-13) and np.isclose(lse[0, i], L, atol=1e-13)


def test_sentence_permutation_equivariance():
    doc = [[3, 5, 2], [4, 1]]
    lv, pa = gen.layout(doc)
    n, H, d = len(lv), 2, 8
    q, k, v, _ = rand_qkv(9, n, H, d)
    o, lse = oracle.forward(*one(lv, pa), q, k, v)
    # swap the first two sentences of section 1: tokens [2..5] (SENT+3) and [6..11] (SENT+5)
    perm = np.concatenate([[0, 1], np.arange(6, 12), np.arange(2, 6), np.arange(12, n)])
    lv2, pa2 = gen.layout([[5, 3, 2], [4, 1]])
    o2, lse2 = oracle.forward(*one(lv2, pa2), q[perm], k[perm], v[perm])
    assert np.allclose(o2, o[perm], atol=1e-13) and np.allclose(lse2, lse[:, perm], atol=1e-13)


def test_pad_rows_and_sequence_isolation():
    b = gen.small_random_batch(31, n_seqs=3, pad_to=80, max_len=70)
    q, k, v, do = rand_qkv(10, b.total_tokens, 2, 8)
    o, lse = oracle.forward(b.level, b.parent, b.cu_seqlens, q, k, v)
    dq, dk, dv = oracle.backward(b.level, b.parent, b.cu_seqlens, q, k, v, do)
    pad = b.level < 0
    assert pad.any()
    assert np.all(o[pad] == 0) and np.all(np.isneginf(lse[:, pad]))
    assert np.all(dq[pad] == 0) and np.all(dk[pad] == 0) and np.all(dv[pad] == 0)
    # each sequence alone gives the same result as inside the batch
    for s in range(b.batch):
        lo, hi = b.cu_seqlens[s], b.cu_seqlens[s + 1]
        o1, lse1 = oracle.forward(*one(b.level[lo:hi], b.parent[lo:hi]), q[lo:hi], k[lo:hi], v[lo:hi])
        assert np.array_equal(o1, o[lo:hi]) and np.array_equal(lse1, lse[:, lo:hi])


# ----------------------------------------------------------------------------------------
# backward
# ----------------------------------------------------------------------------------------
def test_backward_finite_differences():
    b = gen.small_random_batch(41, n_seqs=2, max_len=40, pad_to=None)
    T, H, d = b.total_tokens, 2, 4
    q, k, v, do = rand_qkv(12, T, H, d)
    dq, dk, dv = oracle.backward(b.level, b.parent, b.cu_seqlens, q, k, v, do, scale=0.6)

    def loss(q_, k_, v_):
        o, _ = oracle.forward(b.level, b.parent, b.cu_seqlens, q_, k_, v_, scale=0.6)
        return float((o * do).sum())

    rng = np.random.default_rng(0)
    eps = 1e-6
    real = np.flatnonzero(b.level >= 0)
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(25):
            idx = (int(rng.choice(real)), int(rng.integers(H)), int(rng.integers(d)))
            xp = x.copy(); xp[idx] += eps
            xm = x.copy(); xm[idx] -= eps
            args_p = {"q": (xp, k, v), "k": (q, xp, v), "v": (q, k, xp)}[name]
            args_m = {"q": (xm, k, v), "k": (q, xm, v), "v": (q, k, xm)}[name]
            fd = (loss(*args_p) - loss(*args_m)) / (2 * eps)
            assert abs(fd - g[idx]) < 1e-7 * max(1.0, abs(fd)), (name, idx, fd, g[idx])


def test_backward_dense_textbook_gradient():
    """One-family hierarchy: gradients equal those of dense softmax attention (numpy)."""
    n, H, d = 17, 2, 8
    lv = np.array([0] + [1] * (n - 1), np.int8); pa = np.array([-1] + [0] * (n - 1), np.int32)
    q, k, v, do = rand_qkv(13, n, H, d)
    dq, dk, dv = oracle.backward(*one(lv, pa), q, k, v, do)
    sc = 1 / np.sqrt(d)
    for h in range(H):
        _, _, S = dense_attention_numpy(q[:, h], k[:, h], v[:, h], np.ones((n, n)), sc)
        dP = do[:, h] @ v[:, h].T
        dS = S * (dP - (S * dP).sum(1, keepdims=True))
        assert np.allclose(dv[:, h], S.T @ do[:, h], atol=1e-13)
        assert np.allclose(dq[:, h], sc * dS @ k[:, h], atol=1e-13)
        assert np.allclose(dk[:, h], sc * dS.T @ q[:, h], atol=1e-13)


def test_backward_zero_query_closed_form():
    """Q = 0: S_ij = M_ij/deg(i), so dV_j = sum_i M_ij dO_i / deg(i) and dK = 0."""
    b = gen.small_random_batch(43, n_seqs=2, max_len=80)
    T, H, d = b.total_tokens, 2, 8
    q, k, v, do = rand_qkv(14, T, H, d)
    q[:] = 0
    dq, dk, dv = oracle.backward(b.level, b.parent, b.cu_seqlens, q, k, v, do)
    assert np.allclose(dk, 0, atol=1e-15)
    for s in range(b.batch):
        lo, hi = b.cu_seqlens[s], b.cu_seqlens[s + 1]
        M = oracle.mask(b.level, b.parent, b.cu_seqlens, s).astype(float)
        W = M / np.maximum(M.sum(1, keepdims=True), 1)
        for h in range(H):
            assert np.allclose(dv[lo:hi, h], W.T @ do[lo:hi, h], atol=1e-13)


def test_sampled_rows_and_cols_match_full():
    b = gen.small_random_batch(44, n_seqs=3, max_len=100)
    T, H, d = b.total_tokens, 2, 8
    q, k, v, do = rand_qkv(15, T, H, d)
    o, lse = oracle.forward(b.level, b.parent, b.cu_seqlens, q, k, v)
    dq, dk, dv = oracle.backward(b.level, b.parent, b.cu_seqlens, q, k, v, do)
    idx = np.random.default_rng(1).choice(T, 20, replace=False).astype(np.int32)
    o_r, lse_r, dq_r = oracle.rows(b.level, b.parent, b.cu_seqlens, q, k, v, idx, do=do)
    dk_c, dv_c = oracle.cols(b.level, b.parent, b.cu_seqlens, q, k, v, do, idx)
    assert np.allclose(o_r, o[idx], atol=1e-14) and np.allclose(lse_r, lse[:, idx].T, atol=1e-14, equal_nan=True)
    assert np.allclose(dq_r, dq[idx], atol=1e-13)
    assert np.allclose(dk_c, dk[idx], atol=1e-13) and np.allclose(dv_c, dv[idx], atol=1e-13)


def test_fp32_inputs_are_promoted_exactly():
    b = gen.make_hierarchy(1)
    t = gen.make_tensors(0, b.total_tokens, 1, 64, "f32", names=("q", "k", "v"))
    o32, l32 = oracle.forward(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"])
    o64, l64 = oracle.forward(b.level, b.parent, b.cu_seqlens, *(t[x].astype(np.float64) for x in "qkv"))
    assert np.array_equal(o32, o64) and np.array_equal(l32, l64)


def test_bf16_rounding_helper():
    x = np.array([1.0, 1.00390625, 1.005859375, -3.1415927, 65504.0, 1e-30], np.float32)
    r = gen.round_bf16(x)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: ties go to the even mantissa (1.0)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == np.float32(1.0078125)
    assert np.all(gen.from_bf16_bits(gen.to_bf16_bits(r)) == r)
    assert np.all(np.abs(r - x) <= np.abs(x) * 2.0 ** -8)

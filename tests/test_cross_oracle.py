"""Pins for the cross-attention oracle (decoder rows attending to a level subset of the encoder
tokens of their own document): reductions to library softmax attention, closed forms, finite
differences, invariances."""
import numpy as np
import pytest
from scipy.special import logsumexp, softmax

import gen
from oracle import cross_oracle as co

SEC, SENT, TOK = 1 << 1, 1 << 2, 1 << 3


def batch(seed, n_seqs=3):
    b = gen.small_random_batch(seed, n_seqs=n_seqs, max_len=120, K=(0, 9))
    rng = np.random.default_rng(seed + 100)
    nq = rng.integers(0, 9, size=b.batch)
    nq[0] = max(nq[0], 3)
    cu_q = np.concatenate([[0], np.cumsum(nq)]).astype(np.int32)
    H, d = 2, 8
    qd = rng.standard_normal((int(cu_q[-1]), H, d))
    k, v = (rng.standard_normal((b.total_tokens, H, d)) for _ in range(2))
    do = rng.standard_normal(qd.shape)
    return b, cu_q, qd, k, v, do


def test_hand_counted_subsets():
    # [DOC] [SEC] [SENT] t t [SENT] t [SEC] [SENT] t   +  two PAD tokens
    lv, pa = gen.layout([[2, 1], [1]])
    lv, pa = gen.fit(lv, pa, len(lv) + 2, pad=True)
    cu = np.array([0, len(lv)], np.int32)
    assert [list(s) for s in co.selected(lv, cu, SEC)] == [[1, 7]]
    assert [list(s) for s in co.selected(lv, cu, SEC | SENT)] == [[1, 2, 5, 7, 8]]
    assert [list(s) for s in co.selected(lv, cu, SEC | SENT | TOK)] == [[1, 2, 3, 4, 5, 6, 7, 8, 9]]
    assert [list(s) for s in co.selected(lv, cu, 0xF)] == [list(range(10))]      # PAD never chosen


@pytest.mark.parametrize("mask", [SEC, SEC | SENT, 0xF])
def test_equals_library_softmax_attention_on_the_subset(mask):
    b, cu_q, qd, k, v, _ = batch(1)
    o, lse = co.forward(b.level, b.cu_seqlens, mask, cu_q, qd, k, v)
    for s in range(b.batch):
        lv = b.level[b.cu_seqlens[s]:b.cu_seqlens[s + 1]]
        sel = b.cu_seqlens[s] + np.flatnonzero((lv >= 0) & (((mask >> np.maximum(lv, 0)) & 1) == 1))
        r = slice(cu_q[s], cu_q[s + 1])
        for h in range(2):
            if len(sel) == 0:
                assert np.all(o[r, h] == 0) and np.all(np.isneginf(lse[h, r]))
                continue
            a = qd[r, h] @ k[sel, h].T / np.sqrt(8)
            assert np.allclose(o[r, h], softmax(a, axis=1) @ v[sel, h], atol=1e-13)
            assert np.allclose(lse[h, r], logsumexp(a, axis=1), atol=1e-13)


def test_closed_forms():
    b, cu_q, qd, k, v, do = batch(2, n_seqs=1)
    # zero queries: the plain average of the chosen values, LSE = log(count)
    o, lse = co.forward(b.level, b.cu_seqlens, SEC | SENT, cu_q, np.zeros_like(qd), k, v)
    sel = co.selected(b.level, b.cu_seqlens, SEC | SENT)[0]
    assert np.allclose(o, v[sel].mean(0)[None], atol=1e-14) and np.allclose(lse, np.log(len(sel)))
    # one chosen key ([DOC] only): O = its value, LSE = q.k scale, dQ = 0, dV = sum of dO
    o, lse = co.forward(b.level, b.cu_seqlens, 1, cu_q, qd, k, v)
    assert np.allclose(o, v[0][None], atol=1e-14)
    assert np.allclose(lse.T, (qd * k[0][None]).sum(-1) / np.sqrt(8), atol=1e-13)
    dq, dk, dv = co.backward(b.level, b.cu_seqlens, 1, cu_q, qd, k, v, do)
    assert np.abs(dq).max() < 1e-13 and np.abs(dk).max() < 1e-13
    assert np.allclose(dv[0], do.sum(0), atol=1e-13) and np.abs(dv[1:]).max() == 0


def test_backward_finite_differences_and_zero_outside_subset():
    b, cu_q, qd, k, v, do = batch(3)
    mask = SEC | SENT
    dq, dk, dv = co.backward(b.level, b.cu_seqlens, mask, cu_q, qd, k, v, do)

    def loss(q_, k_, v_):
        return float((co.forward(b.level, b.cu_seqlens, mask, cu_q, q_, k_, v_)[0] * do).sum())
    rng = np.random.default_rng(0)
    eps = 1e-6
    for x, g, idx in ((qd, dq, 0), (k, dk, 1), (v, dv, 2)):
        for _ in range(12):
            i = tuple(int(rng.integers(0, n)) for n in x.shape)
            xp, xm = x.copy(), x.copy()
            xp[i] += eps; xm[i] -= eps
            args_p = [qd, k, v]; args_m = [qd, k, v]
            args_p[idx] = xp; args_m[idx] = xm
            fd = (loss(*args_p) - loss(*args_m)) / (2 * eps)
            assert abs(fd - g[i]) < 1e-6 * max(1.0, abs(fd))
    chosen = np.concatenate(co.selected(b.level, b.cu_seqlens, mask))
    rest = np.setdiff1d(np.arange(b.total_tokens), chosen)
    assert np.all(dk[rest] == 0) and np.all(dv[rest] == 0)


def test_documents_are_isolated_and_key_order_is_irrelevant():
    b, cu_q, qd, k, v, _ = batch(4)
    o, _ = co.forward(b.level, b.cu_seqlens, SEC | SENT | TOK, cu_q, qd, k, v)
    k2, v2 = k.copy(), v.copy()
    s0, s1 = b.cu_seqlens[1], b.cu_seqlens[2]
    k2[s0:s1] += 5.0; v2[s0:s1] -= 3.0                       # disturb document 1 only
    o2, _ = co.forward(b.level, b.cu_seqlens, SEC | SENT | TOK, cu_q, qd, k2, v2)
    keep = np.ones(len(qd), bool); keep[cu_q[1]:cu_q[2]] = False
    assert np.array_equal(o[keep], o2[keep])
    # a one-level list: permuting the chosen tokens (with their K, V rows) leaves O unchanged
    lv = np.array([0] + [1] * 9, np.int8)
    cu = np.array([0, 10], np.int32)
    rng = np.random.default_rng(5)
    q1 = rng.standard_normal((4, 1, 8)); k1 = rng.standard_normal((10, 1, 8)); v1 = rng.standard_normal((10, 1, 8))
    perm = np.concatenate([[0], 1 + rng.permutation(9)])
    oa, _ = co.forward(lv, cu, SEC, np.array([0, 4], np.int32), q1, k1, v1)
    ob, _ = co.forward(lv, cu, SEC, np.array([0, 4], np.int32), q1, k1[perm], v1[perm])
    assert np.allclose(oa, ob, atol=1e-14)

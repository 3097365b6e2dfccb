"""Pins of the positional-encoding oracle: hand-worked index vectors, an independent counter-based
derivation, closed forms, the reduction to the textbook sinusoidal encoding for a one-level list."""
import os

import numpy as np

import gen
from oracle import hpe_oracle as ho
from test_oracle_pins import pvectors as counter_pvectors

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def one(lv, pa):
    return np.asarray(lv, np.int8), np.asarray(pa, np.int32), np.array([0, len(lv)], np.int32)


def test_hand_worked_index_vectors():
    rows = [l.split() for l in open(os.path.join(GOLD, "hand_pvectors_10tok.txt")) if not l.startswith("#")]
    want = np.array([[int(x) for x in r[2:5]] for r in rows])
    lv, pa = gen.layout([[2, 1], [1]])
    assert np.array_equal(ho.pvectors(*one(lv, pa), 3), want)


def test_index_vectors_match_running_counters():
    rng = np.random.default_rng(1)
    for _ in range(50):
        L = int(rng.integers(1, 300))
        lv, pa, _ = gen.gen_fill(rng, L, (1, 4), (1, 4), (0, 9))
        assert np.array_equal(ho.pvectors(*one(lv, pa), 3), counter_pvectors(lv))


def test_root_and_pad_closed_forms():
    lv, pa = gen.fit(*gen.layout([[3, 2]]), 12, pad=True)
    e = ho.hpe(*one(lv, pa), 16, 3)
    assert np.allclose(e[0, 0::2], 0) and np.allclose(e[0, 1::2], 3)     # [DOC]: sin 0 = 0, cos 0 = 1 on 3 levels
    assert np.all(e[lv < 0] == 0)
    # a regular token (1, 1, 2): first pair is sin / cos at w_0 = 1
    t = 4
    assert lv[t] == 3
    assert np.isclose(e[t, 0], np.sin(1) + np.sin(1) + np.sin(2)) and np.isclose(e[t, 1], 2 * np.cos(1) + np.cos(2))


def test_one_level_list_is_the_textbook_sinusoidal_encoding():
    n, d = 40, 32
    lv = np.array([0] + [1] * (n - 1), np.int8); pa = np.array([-1] + [0] * (n - 1), np.int32)
    e = ho.hpe(*one(lv, pa), d, 1)
    pos = np.arange(n)[:, None]                       # child c sits at position c, the root at 0
    div = np.exp(-np.log(10000.0) * np.arange(0, d, 2) / d)[None, :]
    pe = np.zeros((n, d)); pe[:, 0::2] = np.sin(pos * div); pe[:, 1::2] = np.cos(pos * div)
    assert np.allclose(e, pe, atol=1e-12)
    assert np.allclose(e[:, 0::2] ** 2 + e[:, 1::2] ** 2, 1.0)


def test_generic_depth_vectors():
    # root -> a (children a1, a2), b (child b1 -> b11): levels up to 3, numbers by sibling order
    lv, pa = gen.layout_tree([[[], []], [[[]]]])
    want = np.array([[0, 0, 0], [1, 0, 0], [1, 1, 0], [1, 2, 0], [2, 0, 0], [2, 1, 0], [2, 1, 1]])
    assert np.array_equal(ho.pvectors(*one(lv, pa), 3), want)
    assert np.array_equal(ho.pvectors(*one(lv, pa), 2), want[:, :2])

"""Pins of the oracle's search logic (Section 2.2) on hand-worked tables."""
import os

import numpy as np

from oracle import aiq_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "search_hand_tables.txt")


def _table():
    ai, acc, loss = {}, {}, {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#") or line.startswith(("greedy", "coordinate")):
            continue
        q, a, c, l = [f.strip() for f in line.split(":")]
        key = tuple(int(v) for v in q.split())
        ai[key], acc[key], loss[key] = float(a), float(c), float(l)
    return ai, acc, loss


def test_loss_matches_the_hand_table():
    ai, acc, loss = _table()
    assert len(ai) == 9
    for k in ai:
        assert abs(O.aiq_loss(ai[k], acc[k], 1.0, 0.5) - loss[k]) < 1e-12


def test_greedy_and_coordinate_descent_on_the_hand_table():
    ai, acc, _ = _table()
    calls = []

    def acc_fn(schemes):
        calls.append(len(schemes))
        return np.array([acc[tuple(int(v) for v in s)] for s in schemes])

    def ai_fn(s):
        return ai[tuple(int(v) for v in s)]

    q, trace = O.greedy_search(2, acc_fn, ai_fn, 0.5, options=(8, 4))
    assert q.tolist() == [8, 8]
    assert [(t[0], t[1], t[2]) for t in trace] == [(0, 8, 1), (1, 8, 1)]
    assert abs(trace[-1][3] - (-7.5)) < 1e-12
    assert calls == [1, 4, 2]                    # FP32 reference, 4 candidates, then 2

    q, trace = O.coordinate_descent(2, acc_fn, ai_fn, 0.5, options=(32, 8, 4))
    assert q.tolist() == [8, 8]
    assert [(t[0], t[1], t[2]) for t in trace] == [(0, 8, 1), (1, 8, 1), (0, 8, 0), (1, 8, 0)]


def test_greedy_keeps_fp32_when_every_move_hurts():
    def acc_fn(schemes):
        return np.array([1.0 - 0.1 * int(np.sum(s != 32)) for s in schemes])

    def ai_fn(s):
        return 10.0 + float(np.sum(s != 32))

    q, trace = O.greedy_search(3, acc_fn, ai_fn, 0.5)
    assert q.tolist() == [32, 32, 32]
    assert len(trace) == 1 and trace[0][2] == 0
    q, _ = O.coordinate_descent(3, acc_fn, ai_fn, 0.5)
    assert q.tolist() == [32, 32, 32]


def test_greedy_moves_a_layer_at_most_once_and_respects_the_layer_list():
    def acc_fn(schemes):
        return np.ones(len(schemes))

    def ai_fn(s):                                 # lower bits always help; layer 2 helps most
        w = np.array([1.0, 2.0, 4.0, 3.0])
        return float(np.sum(w * (32 - s.astype(np.float64))))

    q, trace = O.greedy_search(4, acc_fn, ai_fn, 0.9, options=(8, 4), layers=[0, 2, 3])
    assert q.tolist() == [4, 32, 4, 4]
    assert [t[0] for t in trace] == [2, 3, 0] and all(t[1] == 4 and t[2] == 1 for t in trace)

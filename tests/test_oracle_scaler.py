"""Pins for the oracle's scaler signals (paper Sec. 4.3.2)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2504_03702_b200 import workloads as W


def state_with_curves(curves, capacity):
    curves = np.asarray(curves, dtype=np.int64)
    s = oracle.State(curves.shape[0], curves.shape[1], capacity, [], [], [], [], 1)
    s.curves[:] = curves
    return s


def test_hand_example():
    """M = 100: overloaded above 95 tokens in more than 10 % of 10 steps (i.e. at least 2 steps);
    idle below 30 tokens throughout."""
    curves = [
        [96, 97, 10, 10, 10, 10, 10, 10, 10, 10],   # 2 hot steps of 10 -> overloaded; max 97
        [96, 95, 95, 10, 10, 10, 10, 10, 10, 10],   # 1 hot step (95 is not above 95) -> not overloaded; max 96
        [29, 29, 0, 0, 0, 0, 0, 0, 0, 0],           # idle throughout; max 29
        [30, 0, 0, 0, 0, 0, 0, 0, 0, 0],            # 30 is not below 30 -> not idle; max 30
    ]
    over, mx, summary = state_with_curves(curves, 100).scaler_signals()
    assert over.tolist() == [2, 1, 0, 0]
    assert mx.tolist() == [97, 96, 29, 30]
    assert summary.tolist() == [1, 3, 97 + 96 + 29 + 30]


def test_all_idle_and_all_hot():
    z = state_with_curves(np.zeros((5, 16)), 1000)
    over, mx, summary = z.scaler_signals()
    assert summary.tolist() == [0, 0, 0] and (over == 0).all()
    h = state_with_curves(np.full((5, 16), 999), 1000)
    over, mx, summary = h.scaler_signals()
    assert summary.tolist() == [5, 5, 5 * 999] and (over == 16).all()


@pytest.mark.parametrize("seed,n_inst,h", [(1, 7, 33), (2, 40, 128), (3, 3, 1), (4, 64, 256)])
def test_matches_exact_rational_enumeration(seed, n_inst, h):
    wl = W.make_random(seed, n_inst, h, 40 * n_inst, 0, max_prompt=400, max_output=2 * h + 3)
    s = oracle.State.from_workload(wl)
    s.anticipate()
    cap = int(np.percentile(s.curves.max(axis=1), 60)) + 1        # some instances above, some below
    s.M = cap
    over, mx, summary = s.scaler_signals()
    hot, idle = Fraction(0.95) * cap, Fraction(0.30) * cap
    want_over = [sum(1 for v in row if Fraction(int(v)) > hot) for row in s.curves]
    want_max = [int(max(row)) for row in s.curves]
    assert over.tolist() == want_over and mx.tolist() == want_max
    assert summary[0] == sum(1 for c in want_over if Fraction(c) > Fraction(0.10) * h)
    assert summary[1] == sum(1 for m in want_max if not Fraction(m) < idle)
    assert summary[2] == sum(want_max)


def test_isolation_count_formula():
    """N_c - sum(max U') / T_f with U' = max_j c / M: four instances at 15 % peak usage -> two can go."""
    s = state_with_curves(np.full((4, 8), 150), 1000)
    _, _, summary = s.scaler_signals()
    assert summary[1] == 0                                   # everyone idle: the action may fire
    assert 4 - summary[2] / (1000 * 0.30) == pytest.approx(2.0)

"""Pins for the oracle's misprediction refinement (paper Sec. 4.3.1, paragraph after the map update)."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2504_03702_b200 import workloads as W
from helpers import brute_curves

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "refine_example.txt")


def load_refine_example(path):
    reqs, built, ticks = [], {}, {}
    for line in open(path):
        line = line.split("#")[0].split()
        if not line:
            continue
        if line[0] == "request":
            reqs.append([int(x) for x in line[1:]])
        elif line[0] == "built":
            built[line[1]] = [int(x) for x in line[2:]]
        elif line[0] == "tick":
            ticks.setdefault(int(line[1]), {})[line[2]] = [int(x) for x in line[3:]]
    return np.array(reqs), built, ticks


def backlog(state):
    n = int(state.n[0])
    live = state.generated[:n] < state.predicted[:n]
    rem = (state.predicted[:n].astype(np.int64) - state.generated[:n])[live]
    return np.bincount(state.instance[:n][live], weights=rem, minlength=state.I).astype(np.int64)


def check_against_definition(state):
    n = int(state.n[0])
    ref = brute_curves(state.prompt[:n], state.generated[:n], state.predicted[:n], state.instance[:n],
                       state.I, state.H)
    np.testing.assert_array_equal(state.curves, ref)
    np.testing.assert_array_equal(state.current_d, backlog(state))


def test_hand_computed_example():
    reqs, built, ticks = load_refine_example(GOLDEN)
    s = oracle.State(1, 8, 1000, reqs[:, 0], reqs[:, 1], reqs[:, 2], reqs[:, 3], len(reqs))
    actual = reqs[:, 4]
    s.anticipate()
    assert s.curves[0].tolist() == built["curve"] and s.current_d.tolist() == built["current_d"]
    for t in sorted(ticks):
        s.step()
        counts = s.refine(actual)
        want = ticks[t]
        assert s.curves[0].tolist() == want["curve"], t
        assert s.current_d.tolist() == want["current_d"], t
        assert s.predicted[:2].tolist() == want["predicted"], t
        assert counts[:2].tolist() == want["counts"], t
    assert s.predicted[:2].tolist() == actual.tolist()


def single(P, g, D, H=64):
    s = oracle.State(1, H, 10 ** 6, [P], [g], [D], [0], 1)
    s.anticipate()
    return s


def test_early_finish_removes_exactly_the_rest_of_the_ramp():
    P, g, D = 37, 4, 19
    s = single(P, g, D)
    total_before = int(s.curves.sum())
    counts = s.refine([g])
    assert counts.tolist() == [1, 0, 0]
    removed = total_before - int(s.curves.sum())
    assert removed == (D - g) * P + (D * (D - 1) - g * (g - 1)) // 2       # sum of P + i for i in [g, D)
    assert not s.curves.any() and s.current_d[0] == 0 and s.predicted[0] == g


def test_early_finish_is_cut_at_the_window():
    P, g, D, H = 11, 2, 40, 8
    s = single(P, g, D, H)
    before = s.curves.copy()
    s.refine([1])                       # reported done (actual <= g)
    assert (before[0] == [P + g + j for j in range(H)]).all()
    assert not s.curves.any() and s.current_d[0] == 0 and s.predicted[0] == g


def test_nothing_happens_while_the_prediction_holds():
    s = single(9, 3, 12)
    before = s.curves.copy()
    for actual in (4, 12, 500):          # still running, and not yet at the predicted end
        assert s.refine([actual]).tolist() == [0, 0, 0]
        np.testing.assert_array_equal(s.curves, before)
        assert s.predicted[0] == 12


@pytest.mark.parametrize("D,want", [(1, 1), (4, 1), (5, 1), (6, 2), (10, 2), (11, 3), (99, 20), (100, 20), (101, 21)])
def test_extension_is_a_fifth_rounded_up(D, want):
    P = 7
    s = oracle.State(1, 64, 10 ** 6, [P], [D], [D], [0], 1)   # at its predicted end: contributes nothing
    s.anticipate()
    assert not s.curves.any()
    counts = s.refine([D + 1000])
    assert counts.tolist() == [0, 1, 0]
    assert want == -(-Fraction(D, 5).numerator // Fraction(D, 5).denominator)       # ceil(D / 5) in exact arithmetic
    assert s.predicted[0] == D + want and s.current_d[0] == want
    row = [P + D + j if j < want else 0 for j in range(64)]
    assert s.curves[0].tolist() == row


def test_repeated_extension_reaches_the_real_length():
    P, D, actual = 3, 10, 57
    s = single(P, 0, D, H=16)
    seen = [D]
    for _ in range(200):
        s.step()
        s.refine([actual])
        check_against_definition(s)
        if s.predicted[0] != seen[-1]:
            seen.append(int(s.predicted[0]))
    # 10 -> 12 -> 15 -> 18 -> 22 -> 27 -> 33 -> 40 -> 48 -> 58, then closed at the real 57
    assert seen == [10, 12, 15, 18, 22, 27, 33, 40, 48, 58, 57]
    assert s.generated[0] == actual and not s.curves.any() and s.current_d[0] == 0


def test_malformed_entries_are_counted_and_skipped():
    s = oracle.State(2, 8, 100, [5, 5, 5], [1, 1, 9], [4, 4, 4], [0, 7, 1], 3)
    s.anticipate()
    before, backlog_before = s.curves.copy(), s.current_d.copy()
    counts = s.refine([0, 3, 3])          # actual < 1; instance out of range; finished long ago (g > D)
    assert counts.tolist() == [0, 0, 2]
    np.testing.assert_array_equal(s.curves, before)
    np.testing.assert_array_equal(s.current_d, backlog_before)


@pytest.mark.parametrize("seed,I,H,n", [(1, 3, 16, 60), (2, 1, 5, 40), (3, 7, 33, 300), (4, 4, 64, 200)])
def test_maps_stay_equal_to_the_definition_on_the_refined_table(seed, I, H, n):
    wl = W.make_random(seed, I, H, n, 0, max_prompt=40, max_output=30)
    err = np.rint((W.Stream(seed, 7).uniform(n) - 0.5) * 40).astype(np.int32)         # real length within 20 tokens
    actual = np.maximum(1, wl.predicted + err).astype(np.int32)                        # some already past their end
    s = oracle.State.from_workload(wl)
    s.anticipate()
    first = s.refine(actual)             # requests whose real end lies behind them close at once
    assert first[0] == int(((actual <= wl.generated) & (wl.generated < wl.predicted)).sum())
    check_against_definition(s)
    total = first.copy()
    for _ in range(int(actual.max()) + 2):
        s.step()
        total += s.refine(actual)
        check_against_definition(s)
    assert not s.curves.any()
    np.testing.assert_array_equal(s.predicted[:n], np.maximum(actual, wl.generated))   # every request ends at its real length
    assert total[2] == 0 and total[0] > 0 and total[1] > 0


def test_refinement_commutes_with_routing_and_steps_on_a_config():
    wl = W.make_config(0)
    table_actual, tick_actual = W.make_actual(wl, W.BASE_SEED)
    s = oracle.State.from_workload(wl)
    s.anticipate()
    ap, ad = wl.ticks[0]
    s.route_batch(ap, ad)
    actual = np.concatenate([table_actual, tick_actual[0]])
    for _ in range(40):
        s.step()
        s.refine(actual)
        check_against_definition(s)


def test_actual_lengths_follow_the_stated_error_model():
    pred = np.full(200000, 2000, np.int32)        # far from the clamps
    act = W.actual_lengths(99, 6, pred)
    err = np.abs(act.astype(np.float64) - pred)
    assert abs(err.mean() - 78.25) < 1.5
    assert abs((err <= 25).mean() - 0.53) < 0.02 and abs((err <= 100).mean() - 0.81) < 0.02
    g = np.arange(200000, dtype=np.int32) % 2100
    assert (W.actual_lengths(99, 6, pred, g) > g).all()

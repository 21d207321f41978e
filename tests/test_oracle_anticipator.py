"""Pins for the oracle's load-look-ahead map (paper Sec. 4.3.1)."""
import os

import numpy as np
import pytest

import oracle
from paper_2504_03702_b200 import workloads as W
from helpers import brute_curves, load_worked_example

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")


def build(prompt, generated, predicted, instance, n_inst, horizon):
    s = oracle.State(n_inst, horizon, 100, prompt, generated, predicted, instance, len(prompt))
    s.anticipate()
    return s


def test_worked_example_curves():
    ex = load_worked_example(GOLDEN)
    req = np.array(ex["request"], dtype=np.int32)
    s = build(req[:, 0], req[:, 1], req[:, 2], req[:, 3], 2, 6)
    assert s.curves[0].tolist() == ex["curve"][0]
    assert s.curves[1].tolist() == ex["curve"][1]
    assert s.current_d.tolist() == ex["current_d"]


@pytest.mark.parametrize("p,d,h", [(10, 5, 16), (3, 1, 4), (100, 16, 16), (7, 40, 16), (0, 3, 5)])
def test_single_ramp_closed_form(p, d, h):
    s = build([p], [0], [d], [0], 1, h)
    c = s.curves[0]
    dc = min(d, h)
    assert c[:dc].tolist() == [p + j for j in range(dc)]          # ramp P, P+1, ...
    assert (c[dc:] == 0).all()                                     # released from step D on
    assert c.sum() == dc * p + dc * (dc - 1) // 2
    assert c.max() == p + dc - 1 and int(np.argmax(c)) == dc - 1   # peak just before release
    assert s.current_d[0] == d                                     # backlog is not cut at H


def test_in_flight_request_is_the_ramp_seen_later():
    full = build([20], [0], [12], [0], 1, 32).curves[0]
    for g in range(12):
        later = build([20], [g], [12], [0], 1, 32).curves[0]
        assert later[: 32 - g].tolist() == full[g:].tolist()


def test_identical_requests_scale_and_instances_are_independent():
    one = build([9], [2], [11], [0], 3, 8).curves
    many = build([9] * 5, [2] * 5, [11] * 5, [1] * 5, 3, 8).curves
    assert (many[1] == 5 * one[0]).all() and (many[0] == 0).all() and (many[2] == 0).all()


def test_finished_and_malformed_requests_contribute_nothing():
    base = build([5, 6], [0, 1], [4, 3], [0, 1], 2, 8)
    more = build([5, 6, 9, 9, 9, 9, -1], [0, 1, 7, 9, 0, -1, 0], [4, 3, 7, 7, 0, 3, 3], [0, 1, 0, 1, 0, 1, 1], 2, 8)
    assert (more.curves == base.curves).all() and (more.current_d == base.current_d).all()
    out = build([5, 6, 9, 9], [0, 1, 0, 0], [4, 3, 5, 5], [0, 1, 2, -1], 2, 8)
    assert (out.curves == base.curves).all()


@pytest.mark.parametrize("seed,n_inst,h,n", [(1, 1, 1, 5), (2, 3, 7, 40), (3, 8, 64, 120), (4, 5, 33, 0),
                                              (5, 2, 100, 60), (6, 16, 4, 200)])
def test_matches_brute_force(seed, n_inst, h, n):
    wl = W.make_random(seed, n_inst, h, n, 0)
    s = oracle.State.from_workload(wl)
    s.anticipate()
    ref = brute_curves(wl.prompt, wl.generated, wl.predicted, wl.instance, n_inst, h)
    assert (s.curves == ref).all()
    live = wl.generated < wl.predicted
    want = np.bincount(wl.instance[live], weights=(wl.predicted - wl.generated)[live], minlength=n_inst)
    assert (s.current_d == want.astype(np.int64)).all()


def test_tiny_config_matches_brute_force():
    wl = W.make_config(0)
    s = oracle.State.from_workload(wl)
    s.anticipate()
    assert (s.curves == brute_curves(wl.prompt, wl.generated, wl.predicted, wl.instance, 8, 64)).all()


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_invariants(idx):
    wl = W.make_config(idx)
    s = oracle.State.from_workload(wl)
    s.anticipate()
    c = s.curves
    n_inst = wl.n_instances
    # step 0 holds every live request's present tokens
    assert c[:, 0].sum() == int(wl.prompt.astype(np.int64).sum() + wl.generated.astype(np.int64).sum())
    # number of requests still running at step j, and its non-increase
    rem = np.minimum(wl.predicted - wl.generated, wl.horizon)
    nact = np.zeros((n_inst, wl.horizon + 1), np.int64)
    np.add.at(nact, (wl.instance, np.zeros_like(rem)), 1)
    np.add.at(nact, (wl.instance, rem), -1)
    nact = np.cumsum(nact, axis=1)[:, : wl.horizon]
    assert (np.diff(nact, axis=1) <= 0).all()
    # between consecutive steps every surviving request grows by one token, released ones drop out
    assert (np.diff(c, axis=1) <= nact[:, 1:]).all()
    aacc = c - nact * np.arange(wl.horizon)[None, :]
    assert (np.diff(aacc, axis=1) <= 0).all() and (aacc >= 0).all()


def test_add_then_subtract_returns_the_map():
    """Early finish (Sec. 4.3.1): subtracting P+i over the steps not run undoes the tail of the ramp."""
    wl = W.make_random(11, 4, 24, 50, 0)
    base = oracle.State.from_workload(wl)
    base.anticipate()
    p, d, true_d, inst = 13, 20, 7, 2
    with_r = build(list(wl.prompt) + [p], list(wl.generated) + [0], list(wl.predicted) + [d],
                   list(wl.instance) + [inst], 4, 24)
    delta = with_r.curves - base.curves
    assert delta[inst].tolist() == [p + j if j < d else 0 for j in range(24)]
    assert (np.delete(delta, inst, axis=0) == 0).all()
    fixed = with_r.curves.copy()
    for j in range(true_d, d):
        fixed[inst, j] -= p + j
    short = build(list(wl.prompt) + [p], list(wl.generated) + [0], list(wl.predicted) + [true_d],
                  list(wl.instance) + [inst], 4, 24)
    assert (fixed == short.curves).all()

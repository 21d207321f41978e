"""Pins for the oracle's load-aware router (paper Sec. 4.3.3) and decode step."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2504_03702_b200 import workloads as W
from helpers import brute_curves, exact_route, load_worked_example

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")


def fresh(wl):
    s = oracle.State.from_workload(wl)
    s.anticipate()
    return s


def test_worked_example_route_and_step():
    ex = load_worked_example(GOLDEN)
    req = np.array(ex["request"], dtype=np.int32)
    s = oracle.State(2, 6, 50, req[:, 0], req[:, 1], req[:, 2], req[:, 3], len(req) + 1)
    s.anticipate()
    score, peak = s.score_all(*ex["arrival"])
    assert peak.tolist() == ex["peak"] and score.tolist() == [float(v) for v in ex["score"]]
    choice, sc = s.route_batch([ex["arrival"][0]], [ex["arrival"][1]])
    assert choice.tolist() == ex["choice"] and sc[0] == float(min(ex["score"]))
    assert s.curves[0].tolist() == ex["curve_after"][0] and s.curves[1].tolist() == ex["curve_after"][1]
    assert s.queued_p.tolist() == ex["queued_p_after"] and s.current_d.tolist() == ex["current_d_after"]
    assert int(s.n[0]) == len(req) + 1 and s.instance[len(req)] == 1 and s.generated[len(req)] == 0
    s.step()
    assert s.curves[0].tolist() == ex["curve_step"][0] and s.curves[1].tolist() == ex["curve_step"][1]
    assert s.current_d.tolist() == ex["current_d_step"] and s.queued_p.tolist() == ex["queued_p_step"]


@pytest.mark.parametrize("seed,n_inst,h,n,a", [(21, 1, 5, 10, 6), (22, 3, 9, 30, 25), (23, 7, 16, 60, 40),
                                                (24, 4, 1, 20, 10), (25, 6, 40, 0, 30)])
def test_matches_exact_rational_router(seed, n_inst, h, n, a):
    wl = W.make_random(seed, n_inst, h, n, a)
    s = fresh(wl)
    c0 = brute_curves(wl.prompt, wl.generated, wl.predicted, wl.instance, n_inst, h)
    assert (s.curves == c0).all()
    ap, ad = wl.ticks[0]
    cd0 = s.current_d.copy()
    choice, score = s.route_batch(ap, ad)
    ch, sc, c1, q1, cd1 = exact_route(c0, np.zeros(n_inst), cd0, ap, ad, wl.capacity_tokens)
    assert choice.tolist() == ch
    for got, want in zip(score, sc):
        assert abs(Fraction(float(got)) - want) <= Fraction(1, 10 ** 12) * max(abs(want), 1)
    assert (s.curves == c1).all() and (s.queued_p == q1).all() and (s.current_d == cd1).all()


def test_exact_router_with_fractional_threshold_and_beta():
    """Capacity not a multiple of 5 and beta != 1: binary64 score against exact rationals, 1e-12 relative."""
    wl = W.make_random(31, 5, 12, 40, 30, capacity=337, beta=0.75)
    s = fresh(wl)
    ap, ad = wl.ticks[0]
    choice, score = s.route_batch(ap, ad)
    ch, sc, c1, _, _ = exact_route(fresh(wl).curves, np.zeros(5), fresh(wl).current_d, ap, ad, 337,
                                   t_mem=Fraction(0.8), beta=Fraction(0.75))
    assert choice.tolist() == ch and (s.curves == c1).all()
    for got, want in zip(score, sc):
        assert abs(Fraction(float(got)) - want) <= Fraction(1, 10 ** 12) * max(abs(want), 1)


def _greedy_least_loaded(load, ap, ad):
    load = [int(v) for v in load]
    out = []
    for p, d in zip(ap, ad):
        i = min(range(len(load)), key=lambda t: (load[t], t))
        load[i] += int(p) + int(d)
        out.append(i)
    return out


@pytest.mark.parametrize("mode", ["beta0", "huge_capacity"])
def test_reduces_to_greedy_least_loaded(mode):
    """Without the memory penalty the score is queued_p + current_d + const: textbook greedy balancing."""
    kw = dict(beta=0.0) if mode == "beta0" else dict(capacity=10 ** 15)
    wl = W.make_random(41, 9, 20, 80, 120, **kw)
    s = fresh(wl)
    start = s.current_d.copy()
    choice, _ = s.route_batch(*wl.ticks[0])
    assert choice.tolist() == _greedy_least_loaded(start, *wl.ticks[0])


def test_single_instance_and_empty_instances():
    wl = W.make_random(42, 1, 8, 12, 9)
    assert fresh(wl).route_batch(*wl.ticks[0])[0].tolist() == [0] * 9
    wl = W.make_random(43, 4, 8, 0, 8, beta=0.0)
    ap = np.full(8, 10, np.int32)
    ad = np.full(8, 5, np.int32)
    assert fresh(wl).route_batch(ap, ad)[0].tolist() == [0, 1, 2, 3, 0, 1, 2, 3]  # ties to the lowest index


def test_winner_score_rises_and_others_do_not_move():
    wl = W.make_random(44, 6, 16, 50, 1)
    s = fresh(wl)
    p, d = int(wl.ticks[0][0][0]), int(wl.ticks[0][1][0])
    before, _ = s.score_all(p, d)
    choice, score = s.route_batch([p], [d])
    after, _ = s.score_all(p, d)
    w = int(choice[0])
    assert score[0] == before.min() and w == int(np.argmin(before))
    assert after[w] >= before[w] + p + d
    assert (np.delete(after, w) == np.delete(before, w)).all()


@pytest.mark.parametrize("idx", [0, 1])
def test_fold_equals_rebuild(idx):
    wl = W.make_config(idx)
    s = fresh(wl)
    s0 = int(s.curves[:, 0].sum())
    choice, _ = s.route_batch(*wl.ticks[0])
    assert int(s.n[0]) == wl.n_requests + wl.n_arrivals
    assert (s.instance[wl.n_requests:] == choice).all()
    rebuilt = oracle.State(wl.n_instances, wl.horizon, wl.capacity_tokens, s.prompt, s.generated,
                           s.predicted, s.instance, len(s.prompt))
    rebuilt.anticipate()
    assert (rebuilt.curves == s.curves).all() and (rebuilt.current_d == s.current_d).all()
    assert int(s.curves[:, 0].sum()) == s0 + int(wl.ticks[0][0].astype(np.int64).sum())
    assert (s.queued_p == np.bincount(choice, weights=wl.ticks[0][0], minlength=wl.n_instances)).all()


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_identity_mode_equals_literal_mode(idx):
    wl = W.make_config(idx)
    a, b = fresh(wl), fresh(wl)
    ca, sa = a.route_batch(*wl.ticks[0])
    cb, sb = b.route_batch(*wl.ticks[0], fast=True)
    assert (ca == cb).all() and (sa == sb).all()
    assert (a.curves == b.curves).all() and (a.queued_p == b.queued_p).all() and (a.instance == b.instance).all()
    # the memory term must really be in play, else the curves would not decide anything
    theta = wl.t_mem * wl.capacity_tokens
    assert (a.curves.max(axis=1) > theta).mean() > 0.2


def test_identity_mode_on_random_shapes():
    for seed, n_inst, h in [(51, 3, 1), (52, 5, 2), (53, 2, 50), (54, 11, 17)]:
        wl = W.make_random(seed, n_inst, h, 40, 60, max_output=70)
        a, b = fresh(wl), fresh(wl)
        ca, sa = a.route_batch(*wl.ticks[0])
        cb, sb = b.route_batch(*wl.ticks[0], fast=True)
        assert (ca == cb).all() and (sa == sb).all() and (a.curves == b.curves).all()


def test_table_full_and_malformed_arrivals():
    wl = W.make_random(61, 3, 8, 10, 6)
    s = oracle.State(3, 8, wl.capacity_tokens, wl.prompt, wl.generated, wl.predicted, wl.instance, 10 + 4)
    s.anticipate()
    choice, _ = s.route_batch(*wl.ticks[0])
    assert (choice[:4] >= 0).all() and (choice[4:] == -1).all() and int(s.n[0]) == 14
    s = fresh(wl)
    ap, ad = wl.ticks[0][0].copy(), wl.ticks[0][1].copy()
    ad[2] = 0
    ap[4] = -3
    choice, _ = s.route_batch(ap, ad)
    assert choice[2] == -1 and choice[4] == -1 and (np.delete(choice, [2, 4]) >= 0).all()
    assert int(s.n[0]) == 10 + 4


# ---------------------------------------------------------------- decode step

def _advance(wl_arrays, k):
    p, g, d, inst = wl_arrays
    return p, np.minimum(g + k, d), d, inst


@pytest.mark.parametrize("seed,n_inst,h", [(71, 3, 6), (72, 5, 16), (73, 2, 1), (74, 4, 80)])
def test_step_equals_rebuild_of_advanced_requests(seed, n_inst, h):
    wl = W.make_random(seed, n_inst, h, 60, 0, max_output=40)
    s = fresh(wl)
    arrays = (wl.prompt, wl.generated, wl.predicted, wl.instance)
    for k in range(1, 45):
        prev = s.curves.copy()
        s.step()
        p, g, d, inst = _advance(arrays, k)
        assert (s.generated[: wl.n_requests] == g).all()
        ref = brute_curves(p, g, d, inst, n_inst, h)
        assert (s.curves == ref).all()
        assert (s.curves[:, :-1] == prev[:, 1:]).all()  # a fixed future step never changes without arrivals
        want = np.bincount(inst, weights=(d - g), minlength=n_inst).astype(np.int64)
        assert (s.current_d == want).all() and (s.queued_p == 0).all()
    assert (s.curves == 0).all() and (s.current_d == 0).all()


def test_step_after_route_on_tiny_config():
    wl = W.make_config(0)
    s = fresh(wl)
    s.route_batch(*wl.ticks[0])
    for _ in range(3):
        s.step()
    n = int(s.n[0])
    ref = brute_curves(s.prompt[:n], s.generated[:n], s.predicted[:n], s.instance[:n], 8, 64)
    assert (s.curves == ref).all()


# ---------------------------------------------------------------- admission of the running-maxima mode on the large configurations

def _clone(s):
    import copy
    return copy.deepcopy(s)


@pytest.mark.slow
def test_identity_mode_on_a_prefix_of_the_large_configuration():
    """The expected values of the largest configuration come from the running-maxima mode (the literal mode
    needs hours there): on its first 512 arrivals the two modes must agree bit for bit."""
    wl = W.make_config(3)
    a = fresh(wl)
    b = _clone(a)
    ap, ad = wl.ticks[0][0][:512], wl.ticks[0][1][:512]
    ca, sa = a.route_batch(ap, ad)
    cb, sb = b.route_batch(ap, ad, fast=True)
    assert (ca == cb).all() and (sa == sb).all()
    assert (a.curves == b.curves).all() and (a.queued_p == b.queued_p).all() and (a.current_d == b.current_d).all()
    assert (a.instance[:int(a.n[0])] == b.instance[:int(b.n[0])]).all()
    # and with the admission queue (levels at which some arrivals of the prefix find every instance overloaded
    # are not reached here: the rule must then route exactly like the plain router, in both modes)
    c, d = _clone(b), _clone(b)
    ap2, ad2 = wl.ticks[0][0][512:768], wl.ticks[0][1][512:768]
    c.make_queue(64)
    d.make_queue(64)
    rc = c.route_admit(ap2, ad2, overload_level=0.95, overload_share=0.10)
    rd = d.route_admit(ap2, ad2, overload_level=0.95, overload_share=0.10, fast=True)
    for x, y in zip(rc, rd):
        assert (np.asarray(x) == np.asarray(y)).all()
    assert (c.curves == d.curves).all() and (c.queue_state == d.queue_state).all()


@pytest.mark.slow
def test_identity_mode_on_the_first_streaming_ticks():
    wl = W.make_config(4, n_ticks=2)
    a = fresh(wl)
    b = _clone(a)
    for ap, ad in wl.ticks:
        a.step()
        b.step()
        ca, sa = a.route_batch(ap, ad)
        cb, sb = b.route_batch(ap, ad, fast=True)
        assert (ca == cb).all() and (sa == sb).all()
    assert (a.curves == b.curves).all() and (a.queued_p == b.queued_p).all() and (a.current_d == b.current_d).all()

"""Pins for the oracle's router on full-width maps (paper Sec. 4.3.1: the map covers the next L
iterations; Sec. 4.3.3: the peak is taken "over the next l iterations")."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2504_03702_b200 import workloads as W
from helpers import brute_curves, exact_route


def fresh(wl):
    s = oracle.State.from_workload(wl)
    s.anticipate()
    return s


@pytest.mark.parametrize("seed,n_inst,width,n,a", [(61, 1, 7, 12, 9), (62, 4, 12, 40, 30), (63, 9, 33, 80, 50)])
def test_window_equal_to_width_is_the_plain_router(seed, n_inst, width, n, a):
    wl = W.make_random(seed, n_inst, width, n, a, max_output=2 * width)
    plain, windowed = fresh(wl), fresh(wl)
    ap, ad = wl.ticks[0]
    c0, s0 = plain.route_batch(ap, ad)
    c1, s1 = windowed.route_window(ap, ad, width)
    assert c0.tolist() == c1.tolist() and s0.tolist() == s1.tolist()
    assert (plain.curves == windowed.curves).all() and (plain.current_d == windowed.current_d).all()
    assert (plain.queued_p == windowed.queued_p).all() and int(plain.n[0]) == int(windowed.n[0])


@pytest.mark.parametrize("seed,n_inst,width,window,n,a", [(64, 3, 10, 3, 30, 25), (65, 6, 24, 5, 60, 40),
                                                          (66, 5, 16, 1, 40, 30), (67, 2, 9, 8, 0, 12)])
def test_matches_exact_rational_router_with_a_window(seed, n_inst, width, window, n, a):
    wl = W.make_random(seed, n_inst, width, n, a, max_output=2 * width)
    s = fresh(wl)
    c0 = brute_curves(wl.prompt, wl.generated, wl.predicted, wl.instance, n_inst, width)
    ap, ad = wl.ticks[0]
    cd0 = s.current_d.copy()
    choice, score = s.route_window(ap, ad, window)
    ch, sc, c1, q1, cd1 = exact_route(c0, np.zeros(n_inst), cd0, ap, ad, wl.capacity_tokens, window=window)
    assert choice.tolist() == ch
    for got, want in zip(score, sc):
        assert abs(Fraction(float(got)) - want) <= Fraction(1, 10 ** 12) * max(abs(want), 1)
    assert (s.curves == c1).all() and (s.queued_p == q1).all() and (s.current_d == cd1).all()


def test_maps_after_routing_equal_a_rebuild_at_full_width():
    """The real update adds the whole ramp, also beyond the window: the maps stay what the
    definition gives for the table with the routed requests in it."""
    wl = W.make_random(68, 5, 40, 70, 45, max_output=90)
    s = fresh(wl)
    ap, ad = wl.ticks[0]
    choice, _ = s.route_window(ap, ad, 6)
    n = int(s.n[0])
    assert n == wl.n_requests + len(ap) and (s.instance[wl.n_requests:n] == choice).all()
    want = brute_curves(s.prompt[:n], s.generated[:n], s.predicted[:n], s.instance[:n], 5, 40)
    assert (s.curves == want).all()
    # and a decode step afterwards is still the shifted rebuild
    s.step()
    g1 = np.minimum(s.generated[:n], s.predicted[:n])
    want = brute_curves(s.prompt[:n], g1, s.predicted[:n], s.instance[:n], 5, 40)
    assert (s.curves == want).all()


def test_a_short_window_does_not_see_a_late_peak():
    """Hand-made: two empty instances but for one long request on instance 0 whose load keeps
    growing.  M = 100, threshold 80.  Arrival (P = 10, D = 8).
    Row 0 = 60 + j for j < 8: with the arrival the peak over all 8 steps is 67 + 17 = 84 > 80, over
    the first 3 steps it is 62 + 12 = 74 < 80.  Row 1 is empty: peak 17 either way.
    Full width: L_0 = 10 + (8 + 8) + 4 = 30, L_1 = 10 + 8 + 0 = 18 -> instance 1.
    With current_d_0 lowered so that the backlog term favours instance 0 the penalty decides:
    take current_d from the table (8 for row 0, 0 for row 1) and add 9 queued tokens on row 1:
    L_1 = 19 + 8 = 27.  Full width: 30 > 27 -> instance 1.  Window 3: L_0 = 26 < 27 -> instance 0."""
    def state():
        s = oracle.State(2, 8, 100, [60], [0], [8], [0], 4)
        s.anticipate()
        s.queued_p[1] = 9
        return s
    full, short = state(), state()
    assert full.curves[0].tolist() == [60 + j for j in range(8)] and int(full.current_d[0]) == 8
    c_full, s_full = full.route_window([10], [8], 8)
    c_short, s_short = short.route_window([10], [8], 3)
    assert c_full.tolist() == [1] and s_full[0] == 27.0
    assert c_short.tolist() == [0] and s_short[0] == 26.0
    assert short.curves[0].tolist() == [60 + j + 10 + j for j in range(8)]

"""Pins for the oracle's router with admission queue (paper Sec. 4.3.3, queueing sentences; overload
criterion of Sec. 4.3.2)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2504_03702_b200 import workloads as W
from helpers import exact_admit


def state_with_curves(curves, capacity, max_requests=64):
    curves = np.asarray(curves, dtype=np.int64)
    s = oracle.State(curves.shape[0], curves.shape[1], capacity, [], [], [], [], max_requests)
    s.curves[:] = curves
    return s


def test_hand_computed_example():
    """I = 2, H = 4, M = 100: overloaded when at least one step (more than 0.10 * 4) is above 95 tokens;
    memory threshold 0.8 * 100 = 80 tokens, beta = 1; queue of one."""
    s = state_with_curves([[96, 10, 10, 10], [50, 50, 50, 50]], 100)
    s.make_queue(1)
    # arrival (46, 2): instance 1 is not overloaded, so it is routed.
    #   instance 0: peak max(96+46, 10+47, 10, 10) = 142 -> L = 46 + 2 + (142 - 80) = 110
    #   instance 1: peak max(50+46, 50+47, 50, 50) =  97 -> L = 46 + 2 + ( 97 - 80) =  65  -> instance 1
    #   instance 1 becomes 96 97 50 50: now every instance has a step above 95.
    # arrival (1, 1): everyone overloaded, joins the queue.  (2, 1), (3, 1): queue full, turned away.
    qc, c, sc = s.route_admit([46, 1, 2, 3], [2, 1, 1, 1])
    assert qc.tolist() == [] and c.tolist() == [1, -2, -3, -3]
    assert sc.tolist() == [65.0, 0.0, 0.0, 0.0]
    assert s.curves.tolist() == [[96, 10, 10, 10], [96, 97, 50, 50]]
    assert s.queue_state.tolist() == [0, 1] and s.queue_items()[0].tolist() == [1]
    assert int(s.n[0]) == 1 and s.queued_p.tolist() == [0, 46] and s.current_d.tolist() == [0, 2]
    # instance 0 drains (as after some decode steps); the waiting request goes first, then the arrival (5, 1).
    s.curves[0] = [10, 10, 10, 10]
    #   waiting (1, 1): instance 0: peak 11 -> L = 1 + 1 = 2; instance 1: peak max(96+1, 97) = 97 -> L = 47 + 3 + 17 = 67
    #   arrival (5, 1): instance 0 (now 11 10 10 10, queued_p 1, current_d 1): peak 16 -> L = 6 + 2 = 8;
    #                   instance 1: peak max(96+5, 97) = 101 -> L = 51 + 3 + 21 = 75
    qc, c, sc = s.route_admit([5], [1])
    assert qc.tolist() == [0] and c.tolist() == [0] and sc.tolist() == [8.0]
    assert s.curves[0].tolist() == [16, 10, 10, 10]
    assert s.queue_state.tolist() == [0, 0]          # head moved on by one, modulo the capacity of one


@pytest.mark.parametrize("idx", [0, 1])
def test_never_overloaded_is_the_plain_router(idx):
    wl = W.make_config(idx)
    a, b = oracle.State.from_workload(wl), oracle.State.from_workload(wl)
    a.anticipate(); b.anticipate()
    a.make_queue(8)
    ap, ad = wl.ticks[0]
    qc, c, sc = a.route_admit(ap, ad, overload_level=1e9)
    wc, ws = b.route_batch(ap, ad)
    assert (c == wc).all() and (sc == ws).all() and len(qc) == 0
    assert (a.curves == b.curves).all() and (a.current_d == b.current_d).all() and a.queue_state.tolist() == [0, 0]


def test_everyone_overloaded_from_the_start_queues_then_turns_away():
    wl = W.make_random(3, 4, 8, 40, 10)
    s = oracle.State.from_workload(wl)
    s.anticipate()
    before = s.curves.copy()
    s.make_queue(4)
    ap, ad = wl.ticks[0]
    qc, c, sc = s.route_admit(ap, ad, overload_level=-1.0)      # every step of every map is "above"
    assert c.tolist() == [-2] * 4 + [-3] * 6 and not sc.any()
    assert (s.curves == before).all() and int(s.n[0]) == 40
    assert s.queue_items()[0].tolist() == ap[:4].tolist() and s.queue_items()[1].tolist() == ad[:4].tolist()
    # still blocked: the waiting ones keep their places, a new arrival is turned away
    qc, c, _ = s.route_admit(ap[:1], ad[:1], overload_level=-1.0)
    assert qc.tolist() == [-2] * 4 and c.tolist() == [-3] and s.queue_state.tolist() == [0, 4]


@pytest.mark.parametrize("seed,I,H,n,a,qcap,level", [(11, 3, 8, 30, 40, 5, 0.7), (12, 2, 5, 10, 30, 0, 0.7),
                                                     (13, 5, 16, 80, 60, 100, 0.5), (14, 1, 4, 6, 12, 3, 0.9),
                                                     (15, 4, 12, 50, 64, 7, 0.7)])
def test_against_exact_arithmetic_over_several_calls(seed, I, H, n, a, qcap, level):
    wl = W.make_random(seed, I, H, n, a, max_prompt=30, max_output=20)
    s = oracle.State.from_workload(wl)
    s.anticipate()
    s.make_queue(qcap)
    ap, ad = wl.ticks[0]
    share = 0.25
    blocked_seen = routed_seen = False
    for call in range(4):
        lo, hi = call * a // 4, (call + 1) * a // 4
        waiting = list(zip(*[x.tolist() for x in s.queue_items()]))
        want = exact_admit(s.curves, s.queued_p, s.current_d, waiting, list(zip(ap[lo:hi].tolist(), ad[lo:hi].tolist())),
                           s.M, qcap, Fraction(str(level)), Fraction(str(share)))   # the decimal thresholds, exactly
        qc, c, _ = s.route_admit(ap[lo:hi], ad[lo:hi], overload_level=level, overload_share=share)
        assert qc.tolist() == want[0] and c.tolist() == want[1]
        got_queue = list(zip(*[x.tolist() for x in s.queue_items()]))
        assert got_queue == want[2]
        assert (s.curves == want[3]).all() and (s.queued_p == want[4]).all() and (s.current_d == want[5]).all()
        blocked_seen |= -2 in c.tolist() or -3 in c.tolist()
        routed_seen |= any(v >= 0 for v in c.tolist())
        for _ in range(3):        # a few decode steps drain the maps between calls
            s.step()
    assert routed_seen and blocked_seen


@pytest.mark.parametrize("idx,level", [(0, 0.9), (1, 1.0), (2, 1.1)])
def test_running_counts_mode_equals_literal_mode(idx, level):
    wl = W.make_config(idx, scale=0.25 if idx == 2 else 1.0)
    a, b = oracle.State.from_workload(wl), oracle.State.from_workload(wl)
    a.anticipate(); b.anticipate()
    a.make_queue(50); b.make_queue(50)
    ap, ad = wl.ticks[0]
    half = len(ap) // 2
    for lo, hi in ((0, half), (half, len(ap))):
        ra = a.route_admit(ap[lo:hi], ad[lo:hi], overload_level=level, overload_share=0.05)
        rb = b.route_admit(ap[lo:hi], ad[lo:hi], overload_level=level, overload_share=0.05, fast=True)
        for x, y in zip(ra, rb):
            assert (x == y).all()
        assert (a.curves == b.curves).all() and (a.queue_state == b.queue_state).all()
        assert (a.queue_prompt == b.queue_prompt).all()
        for _ in range(20):
            a.step(); b.step()


def test_ring_wraps_and_keeps_order():
    """Capacity 3, calls alternate between blocked and free: the head walks around the ring."""
    s = state_with_curves([[0, 0, 0, 0]], 100, max_requests=64)
    s.make_queue(3)
    order = []
    nxt = 1
    for rnd in range(5):
        s.curves[0] = [99, 99, 99, 99]                       # overloaded: arrivals wait
        qc, c, _ = s.route_admit([nxt, nxt + 1], [1, 1])
        nxt += 2
        assert all(v == -2 for v in qc)
        s.curves[0] = [0, 0, 0, 0]                           # free again, room for exactly two more cells above 95? no: all routed
        s.queued_p[:] = 0
        waiting = s.queue_items()[0].tolist()
        qc, c, _ = s.route_admit([], [])
        assert qc.tolist() == [0] * len(waiting) and s.queue_state[1] == 0
        order += waiting
    n = int(s.n[0])
    assert s.prompt[:n].tolist() == order                   # routed in arrival order
    assert order == [1, 2, 3, 4, 5, 6, 7, 8, 9, 10]
    assert 0 <= s.queue_state[0] < 3


def test_malformed_and_full_table():
    s = state_with_curves([[0, 0], [0, 0]], 100, max_requests=2)
    s.make_queue(4)
    qc, c, _ = s.route_admit([5, -1, 6, 7, 8], [1, 1, 0, 1, 1])
    assert c.tolist() == [0, -1, -1, 1, -1]                  # malformed ones dropped; the table holds two requests
    assert int(s.n[0]) == 2 and s.queue_state.tolist() == [0, 0]

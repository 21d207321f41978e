"""CPU oracle (test infrastructure only): ctypes front of preserve_oracle.cpp.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may
import this package.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .build import build as _build

_lib = None


def _p(a: np.ndarray, ty):
    return a.ctypes.data_as(C.POINTER(ty))


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build())
        i32p, i64p, f64p = C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.POINTER(C.c_double)
        _lib.orc_anticipate.argtypes = [i32p, i32p, i32p, i32p, C.c_int64, C.c_int32, C.c_int32, i64p, i64p]
        _lib.orc_anticipate.restype = None
        route_args = [i32p, i32p, C.c_int64, C.c_int32, C.c_int32, C.c_int64, C.c_double, C.c_double,
                      i64p, i64p, i64p, i32p, i32p, i32p, i32p, i64p, C.c_int64, i32p, f64p]
        for fn in (_lib.orc_route_batch, _lib.orc_route_batch_fast):
            fn.argtypes = route_args
            fn.restype = C.c_int64
        _lib.orc_route_window.argtypes = [i32p, i32p, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_double,
                                          C.c_double, i64p, i64p, i64p, i32p, i32p, i32p, i32p, i64p, C.c_int64, i32p,
                                          f64p]
        _lib.orc_route_window.restype = C.c_int64
        _lib.orc_score_all.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_double,
                                       C.c_double, i64p, i64p, i64p, f64p, i64p]
        _lib.orc_score_all.restype = None
        _lib.orc_scaler_signals.argtypes = [i64p, C.c_int32, C.c_int32, C.c_int64, C.c_double, C.c_double,
                                            C.c_double, i32p, i64p, i64p]
        _lib.orc_scaler_signals.restype = None
        _lib.orc_route_admit.argtypes = [i32p, i32p, C.c_int64, C.c_int32, C.c_int32, C.c_int64, C.c_double, C.c_double,
                                         C.c_double, C.c_double, i32p, i32p, i64p, C.c_int64, i32p,
                                         i64p, i64p, i64p, i32p, i32p, i32p, i32p, i64p, C.c_int64, i32p, f64p,
                                         C.c_int32]
        _lib.orc_route_admit.restype = None
        _lib.orc_refine.argtypes = [i32p, i32p, i32p, i32p, i32p, C.c_int64, C.c_int32, C.c_int32, i64p, i64p, i64p]
        _lib.orc_refine.restype = None
        _lib.orc_step.argtypes = [i32p, i32p, i32p, i32p, C.c_int64, C.c_int32, C.c_int32, i64p, i64p, i64p]
        _lib.orc_step.restype = None
    return _lib


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


class State:
    """Host-side mirror of everything the path reads and writes."""

    def __init__(self, n_instances, horizon, capacity_tokens, prompt, generated, predicted, instance,
                 max_requests, t_mem=0.8, beta=1.0):
        self.I, self.H, self.M = int(n_instances), int(horizon), int(capacity_tokens)
        self.t_mem, self.beta = float(t_mem), float(beta)
        n = len(prompt)
        self.max_requests = int(max(max_requests, n, 1))
        self.prompt = np.zeros(self.max_requests, np.int32)
        self.generated = np.zeros(self.max_requests, np.int32)
        self.predicted = np.zeros(self.max_requests, np.int32)
        self.instance = np.zeros(self.max_requests, np.int32)
        self.prompt[:n], self.generated[:n] = _i32(prompt), _i32(generated)
        self.predicted[:n], self.instance[:n] = _i32(predicted), _i32(instance)
        self.n = np.array([n], np.int64)
        self.curves = np.zeros((self.I, self.H), np.int64)
        self.queued_p = np.zeros(self.I, np.int64)
        self.current_d = np.zeros(self.I, np.int64)

    @classmethod
    def from_workload(cls, wl):
        return cls(wl.n_instances, wl.horizon, wl.capacity_tokens, wl.prompt, wl.generated, wl.predicted,
                   wl.instance, wl.max_requests, wl.t_mem, wl.beta)

    def anticipate(self):
        lib().orc_anticipate(_p(self.prompt, C.c_int32), _p(self.generated, C.c_int32),
                             _p(self.predicted, C.c_int32), _p(self.instance, C.c_int32),
                             int(self.n[0]), self.I, self.H, _p(self.curves, C.c_int64),
                             _p(self.current_d, C.c_int64))

    def route_batch(self, arr_prompt, arr_predicted, fast=False, want_score=True):
        ap, ad = _i32(arr_prompt), _i32(arr_predicted)
        a = len(ap)
        choice = np.full(a, -1, np.int32)
        score = np.zeros(a, np.float64)
        fn = lib().orc_route_batch_fast if fast else lib().orc_route_batch
        fn(_p(ap, C.c_int32), _p(ad, C.c_int32), a, self.I, self.H, self.M, self.t_mem, self.beta,
           _p(self.curves, C.c_int64), _p(self.queued_p, C.c_int64), _p(self.current_d, C.c_int64),
           _p(self.prompt, C.c_int32), _p(self.generated, C.c_int32), _p(self.predicted, C.c_int32),
           _p(self.instance, C.c_int32), _p(self.n, C.c_int64), self.max_requests,
           _p(choice, C.c_int32), _p(score, C.c_double) if want_score else None)
        return choice, score

    def route_window(self, arr_prompt, arr_predicted, window, want_score=True):
        """Router on full-width maps: the state's horizon is the map width L, peaks are taken over
        the first `window` iterations, the real update adds the whole ramp."""
        ap, ad = _i32(arr_prompt), _i32(arr_predicted)
        a = len(ap)
        choice = np.full(a, -1, np.int32)
        score = np.zeros(a, np.float64)
        lib().orc_route_window(_p(ap, C.c_int32), _p(ad, C.c_int32), a, self.I, self.H, int(window), self.M,
                               self.t_mem, self.beta, _p(self.curves, C.c_int64), _p(self.queued_p, C.c_int64),
                               _p(self.current_d, C.c_int64), _p(self.prompt, C.c_int32),
                               _p(self.generated, C.c_int32), _p(self.predicted, C.c_int32),
                               _p(self.instance, C.c_int32), _p(self.n, C.c_int64), self.max_requests,
                               _p(choice, C.c_int32), _p(score, C.c_double) if want_score else None)
        return choice, score

    def make_queue(self, capacity):
        """Empty admission queue (ring) of the given capacity."""
        self.queue_capacity = int(capacity)
        self.queue_prompt = np.zeros(max(self.queue_capacity, 1), np.int32)
        self.queue_predicted = np.zeros(max(self.queue_capacity, 1), np.int32)
        self.queue_state = np.zeros(2, np.int64)       # head, length

    def queue_items(self):
        """Waiting requests, oldest first, as (prompt, predicted) arrays."""
        head, n = (int(v) for v in self.queue_state)
        idx = (head + np.arange(n)) % max(self.queue_capacity, 1)
        return self.queue_prompt[idx].copy(), self.queue_predicted[idx].copy()

    def route_admit(self, arr_prompt, arr_predicted, overload_level=0.95, overload_share=0.10, fast=False,
                    want_score=True):
        """Router with the admission queue. Returns (queue_choice, choice, score)."""
        ap, ad = _i32(arr_prompt), _i32(arr_predicted)
        a = len(ap)
        waiting = int(self.queue_state[1])
        qchoice = np.full(max(waiting, 1), -9, np.int32)
        choice = np.full(max(a, 1), -9, np.int32)
        score = np.zeros(max(a, 1), np.float64)
        lib().orc_route_admit(_p(ap, C.c_int32), _p(ad, C.c_int32), a, self.I, self.H, self.M, self.t_mem,
                              self.beta, float(overload_level), float(overload_share),
                              _p(self.queue_prompt, C.c_int32), _p(self.queue_predicted, C.c_int32),
                              _p(self.queue_state, C.c_int64), self.queue_capacity, _p(qchoice, C.c_int32),
                              _p(self.curves, C.c_int64), _p(self.queued_p, C.c_int64), _p(self.current_d, C.c_int64),
                              _p(self.prompt, C.c_int32), _p(self.generated, C.c_int32),
                              _p(self.predicted, C.c_int32), _p(self.instance, C.c_int32), _p(self.n, C.c_int64),
                              self.max_requests, _p(choice, C.c_int32), _p(score, C.c_double) if want_score else None,
                              1 if fast else 0)
        return qchoice[:waiting], choice[:a], score[:a]

    def score_all(self, p, d):
        score = np.zeros(self.I, np.float64)
        peak = np.zeros(self.I, np.int64)
        lib().orc_score_all(int(p), int(d), self.I, self.H, self.M, self.t_mem, self.beta,
                            _p(self.curves, C.c_int64), _p(self.queued_p, C.c_int64),
                            _p(self.current_d, C.c_int64), _p(score, C.c_double), _p(peak, C.c_int64))
        return score, peak

    def step(self):
        lib().orc_step(_p(self.prompt, C.c_int32), _p(self.generated, C.c_int32),
                       _p(self.predicted, C.c_int32), _p(self.instance, C.c_int32), int(self.n[0]),
                       self.I, self.H, _p(self.curves, C.c_int64), _p(self.queued_p, C.c_int64),
                       _p(self.current_d, C.c_int64))

    def refine(self, actual):
        """Misprediction refinement against the real lengths `actual` (one per table row in use).
        Returns counts int64[3] = (early finishes, extensions, malformed entries)."""
        n = int(self.n[0])
        act = _i32(actual)
        assert len(act) >= n
        counts = np.zeros(3, np.int64)
        lib().orc_refine(_p(self.prompt, C.c_int32), _p(self.generated, C.c_int32), _p(self.predicted, C.c_int32),
                         _p(self.instance, C.c_int32), _p(act, C.c_int32), n, self.I, self.H,
                         _p(self.curves, C.c_int64), _p(self.current_d, C.c_int64), _p(counts, C.c_int64))
        return counts

    def scaler_signals(self, overload_level=0.95, overload_share=0.10, idle_level=0.30):
        """Returns (over_count int32[I], row_max int64[I], summary int64[3])."""
        over = np.zeros(self.I, np.int32)
        mx = np.zeros(self.I, np.int64)
        summary = np.zeros(3, np.int64)
        lib().orc_scaler_signals(_p(self.curves, C.c_int64), self.I, self.H, self.M, float(overload_level),
                                 float(overload_share), float(idle_level), _p(over, C.c_int32),
                                 _p(mx, C.c_int64), _p(summary, C.c_int64))
        return over, mx, summary

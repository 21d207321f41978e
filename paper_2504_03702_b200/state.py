"""Device-resident state of the path: thin holder of the tensors the C-ABI calls act on.

This is plumbing (torch allocates device memory and provides the stream); each method is
one C-ABI call.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


class DeviceState:
    # which routing kernel new states select (B.ROUTE_AUTO leaves the library's choice)
    default_router = B.ROUTE_AUTO

    def __init__(self, n_instances, horizon, capacity_tokens, max_requests, t_mem=0.8, beta=1.0,
                 device="cuda:0"):
        self.I, self.H = int(n_instances), int(horizon)
        self.capacity_tokens, self.t_mem, self.beta = int(capacity_tokens), float(t_mem), float(beta)
        self.max_requests = int(max_requests)
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            code, self.ctx = B.pre_create(n_instances, horizon, capacity_tokens, t_mem, beta, max_requests)
        B.check(code, "pre_create")
        if DeviceState.default_router != B.ROUTE_AUTO:
            B.check(B.pre_route_select(self.ctx, DeviceState.default_router), "pre_route_select")
        i32 = dict(dtype=torch.int32, device=self.device)
        i64 = dict(dtype=torch.int64, device=self.device)
        self.prompt = torch.zeros(self.max_requests, **i32)
        self.generated = torch.zeros(self.max_requests, **i32)
        self.predicted = torch.zeros(self.max_requests, **i32)
        self.instance = torch.zeros(self.max_requests, **i32)
        self.n_requests = torch.zeros(1, **i64)
        self.curves = torch.zeros(self.I, self.H, **i64)
        self.queued_p = torch.zeros(self.I, **i64)
        self.current_d = torch.zeros(self.I, **i64)

    @classmethod
    def from_workload(cls, wl, device="cuda:0"):
        st = cls(wl.n_instances, wl.horizon, wl.capacity_tokens, max(wl.max_requests, 1), wl.t_mem, wl.beta,
                 device)
        st.load_requests(wl.prompt, wl.generated, wl.predicted, wl.instance)
        return st

    def load_requests(self, prompt, generated, predicted, instance):
        n = len(prompt)
        for dst, src in ((self.prompt, prompt), (self.generated, generated), (self.predicted, predicted),
                         (self.instance, instance)):
            dst[:n].copy_(torch.as_tensor(np.ascontiguousarray(src, dtype=np.int32)))
        self.n_requests.fill_(n)
        self.n_host = n

    def anticipate(self, n_requests=None):
        n = self.n_host if n_requests is None else int(n_requests)
        B.check(B.pre_anticipate(self.ctx, self.prompt, self.generated, self.predicted, self.instance, n,
                                 self.curves, self.current_d), "pre_anticipate")

    def route_batch(self, arr_prompt, arr_predicted, want_score=True):
        """arr_* are int32 device tensors. Returns (choice int32[A], score float64[A] or None) on device."""
        a = int(arr_prompt.shape[0])
        choice = torch.empty(a, dtype=torch.int32, device=self.device)
        score = torch.empty(a, dtype=torch.float64, device=self.device) if want_score else None
        B.check(B.pre_route_batch(self.ctx, arr_prompt, arr_predicted, a, self.curves, self.queued_p,
                                  self.current_d, self.prompt, self.generated, self.predicted, self.instance,
                                  self.n_requests, choice, score), "pre_route_batch")
        return choice, score

    def make_queue(self, capacity):
        """Empty admission queue (a ring in device memory) of the given capacity."""
        self.queue_capacity = int(capacity)
        n = max(self.queue_capacity, 1)
        self.queue_prompt = torch.zeros(n, dtype=torch.int32, device=self.device)
        self.queue_predicted = torch.zeros(n, dtype=torch.int32, device=self.device)
        self.queue_choice = torch.zeros(n, dtype=torch.int32, device=self.device)
        self.queue_state = torch.zeros(2, dtype=torch.int64, device=self.device)     # head, length

    def route_admit(self, arr_prompt, arr_predicted, overload_level=0.95, overload_share=0.10, want_score=True):
        """Router with the admission queue. Returns device tensors (queue_choice int32[capacity],
        choice int32[A], score float64[A] or None); queue_choice is meaningful for the entries that
        were waiting when the call was made."""
        a = int(arr_prompt.shape[0])
        choice = torch.empty(a, dtype=torch.int32, device=self.device)
        score = torch.empty(a, dtype=torch.float64, device=self.device) if want_score else None
        B.check(B.pre_route_admit(self.ctx, arr_prompt, arr_predicted, a, overload_level, overload_share,
                                  self.queue_prompt, self.queue_predicted, self.queue_state, self.queue_capacity,
                                  self.queue_choice, self.curves, self.queued_p, self.current_d, self.prompt,
                                  self.generated, self.predicted, self.instance, self.n_requests, choice, score),
                "pre_route_admit")
        return self.queue_choice, choice, score

    def step(self):
        B.check(B.pre_step(self.ctx, self.prompt, self.generated, self.predicted, self.instance,
                           self.n_requests, self.curves, self.queued_p, self.current_d), "pre_step")

    def refine(self, actual, want_counts=True):
        """`actual`: device int32 tensor of real response lengths, one per table row in use.
        Returns the device tensor int64[3] (early finishes, extensions, malformed rows) or None."""
        counts = torch.empty(3, dtype=torch.int64, device=self.device) if want_counts else None
        B.check(B.pre_refine(self.ctx, self.prompt, self.generated, self.predicted, self.instance, actual,
                             self.n_requests, self.curves, self.current_d, counts), "pre_refine")
        return counts

    def scaler_signals(self, overload_level=0.95, overload_share=0.10, idle_level=0.30):
        """Returns device tensors (over_count int32[I], row_max int64[I], summary int64[3])."""
        over = torch.empty(self.I, dtype=torch.int32, device=self.device)
        row_max = torch.empty(self.I, dtype=torch.int64, device=self.device)
        summary = torch.empty(3, dtype=torch.int64, device=self.device)
        B.check(B.pre_scaler_signals(self.ctx, self.curves, overload_level, overload_share, idle_level, over,
                                     row_max, summary), "pre_scaler_signals")
        return over, row_max, summary

    def tick(self, actual=None, signals=True, overload_level=0.95, overload_share=0.10, idle_level=0.30):
        """pre_tick: decode step, refinement against `actual` (if given) and scaler signals (if wanted) in one call.
        Returns (counts int64[3] or None, over_count, row_max, summary) as device tensors (None where not asked)."""
        counts = torch.empty(3, dtype=torch.int64, device=self.device) if actual is not None else None
        over = row_max = summary = None
        if signals:
            over = torch.empty(self.I, dtype=torch.int32, device=self.device)
            row_max = torch.empty(self.I, dtype=torch.int64, device=self.device)
            summary = torch.empty(3, dtype=torch.int64, device=self.device)
        B.check(B.pre_tick(self.ctx, self.prompt, self.generated, self.predicted, self.instance, actual,
                           self.n_requests, self.curves, self.queued_p, self.current_d, overload_level,
                           overload_share, idle_level, over, row_max, summary, counts), "pre_tick")
        return counts, over, row_max, summary

    # ---- full-width maps kept as a ring (the state's own maps are then the window of width H = l)

    def make_ring(self, width, builder=None):
        """Allocates ring[I][width] and the head word, and builds the full-width maps from the table
        (pre_anticipate on a context of horizon `width`; pass one as `builder` to reuse it)."""
        self.width = int(width)
        self.ring = torch.zeros(self.I, self.width, dtype=torch.int64, device=self.device)
        self.head = torch.zeros(1, dtype=torch.int64, device=self.device)
        own = builder is None
        if own:
            with torch.cuda.device(self.device):
                code, builder = B.pre_create(self.I, self.width, self.capacity_tokens, self.t_mem, self.beta,
                                             self.max_requests)
            B.check(code, "pre_create")
        B.check(B.pre_anticipate(builder, self.prompt, self.generated, self.predicted, self.instance, self.n_host,
                                 self.ring, self.current_d), "pre_anticipate")
        if own:
            torch.cuda.synchronize(self.device)
            B.pre_destroy(builder)

    def ring_window(self):
        B.check(B.pre_ring_window(self.ctx, self.ring, self.width, self.head, self.curves), "pre_ring_window")

    def ring_fold(self, arr_prompt, arr_predicted, choice):
        B.check(B.pre_ring_fold(self.ctx, arr_prompt, arr_predicted, choice, int(arr_prompt.shape[0]), self.ring,
                                self.width, self.head), "pre_ring_fold")

    def ring_step(self):
        B.check(B.pre_ring_step(self.ctx, self.prompt, self.generated, self.predicted, self.instance,
                                self.n_requests, self.ring, self.width, self.head, self.queued_p, self.current_d),
                "pre_ring_step")

    def ring_refine(self, actual, want_counts=True):
        """pre_refine on the ring; returns the device tensor int64[3] of counts or None."""
        counts = torch.empty(3, dtype=torch.int64, device=self.device) if want_counts else None
        B.check(B.pre_ring_refine(self.ctx, self.prompt, self.generated, self.predicted, self.instance, actual,
                                  self.n_requests, self.ring, self.width, self.head, self.current_d, counts),
                "pre_ring_refine")
        return counts

    def ring_logical(self):
        """The ring read out in logical order (column j = j iterations from now); synchronises."""
        h = int(self.head.item())
        idx = (h + torch.arange(self.width, device=self.device)) % self.width
        return self.ring[:, idx]

    def status(self):
        return B.pre_status(self.ctx)

    def select_router(self, path):
        """B.ROUTE_AUTO, B.ROUTE_SCAN or B.ROUTE_SUMMARY: which kernel routes the batches (same results)."""
        B.check(B.pre_route_select(self.ctx, path), "pre_route_select")

    def sync_count(self):
        """Reads the device-side request count back (synchronises)."""
        self.n_host = int(self.n_requests.item())
        return self.n_host

    def close(self):
        if getattr(self, "ctx", None):
            torch.cuda.synchronize(self.device)
            B.pre_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

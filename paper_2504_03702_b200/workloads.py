"""Seeded synthetic workloads for the load anticipator and the load-aware router.

This module only draws numbers.  It holds none of the method's arithmetic (no
curve, peak or score is computed here) so that both the CUDA path and the
CPU oracle can be fed the very same arrays.

The inputs stand in for the serving traces the paper evaluates on (an Azure
inference trace and ShareGPT conversations, Evaluation Setup / Workloads):
those are not redistributable here, so request lengths are drawn from clamped
log-normal distributions and instance assignment is uniform or Zipf.

Everything is derived from a counter-based SplitMix64 stream (Steele, Lea &
Flood, "Fast splittable pseudorandom number generators", OOPSLA 2014) and from
transforms written out below, so the arrays do not depend on a library's
distribution code.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

BASE_SEED = 250403702


def _mix(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function on an array of uint64 states."""
    z = z.copy()
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


class Stream:
    """Counter-based generator: element i of stream s is mix(key(seed, s) + (i+1)*golden)."""

    def __init__(self, seed: int, stream: int):
        with np.errstate(over="ignore"):
            k = np.array([np.uint64(seed)], dtype=np.uint64) * _GOLDEN + np.array(
                [np.uint64(stream)], dtype=np.uint64
            ) * _M1
            self._key = _mix(k)[0]
        self._pos = 0

    def raw(self, n: int) -> np.ndarray:
        with np.errstate(over="ignore"):
            ctr = np.arange(self._pos + 1, self._pos + n + 1, dtype=np.uint64)
            out = _mix(self._key + ctr * _GOLDEN)
        self._pos += n
        return out

    def uniform(self, n: int) -> np.ndarray:
        """Doubles in [0, 1) with 53 random bits."""
        return (self.raw(n) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)

    def normal(self, n: int) -> np.ndarray:
        """Standard normals by the Box-Muller transform (cosine branch)."""
        u1 = 1.0 - self.uniform(n)  # (0, 1]
        u2 = self.uniform(n)
        return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)

    def lognormal_int(self, n: int, median: float, sigma: float, lo: int, hi: int) -> np.ndarray:
        x = np.rint(np.exp(np.log(median) + sigma * self.normal(n)))
        return np.clip(x, lo, hi).astype(np.int32)

    def poisson(self, lam: float) -> int:
        """Count of unit-rate exponential inter-arrival times that fit in [0, lam)."""
        m = int(lam + 12.0 * np.sqrt(lam) + 32)
        gaps = -np.log(1.0 - self.uniform(m))
        t = np.cumsum(gaps)
        assert t[-1] > lam, "poisson draw ran out of exponentials"
        return int(np.searchsorted(t, lam, side="left"))


@dataclass
class Workload:
    """One seeded configuration: the in-flight request table and the arrivals to route."""

    name: str
    n_instances: int                 # I
    horizon: int                     # H (the paper's look-ahead l)
    prompt: np.ndarray               # int32[N]  P
    generated: np.ndarray            # int32[N]  g, tokens generated so far
    predicted: np.ndarray            # int32[N]  D, predicted output length
    instance: np.ndarray             # int32[N]  instance the request runs on
    capacity_tokens: int             # M, KV token capacity of an instance
    t_mem: float = 0.8
    beta: float = 1.0
    # one entry per scheduler tick: (arrival prompt, arrival predicted); a
    # one-shot batch configuration has exactly one entry and no decode step.
    ticks: List[Tuple[np.ndarray, np.ndarray]] = field(default_factory=list)
    streaming: bool = False          # True: each tick is "step, then route"
    max_requests: int = 0

    @property
    def n_requests(self) -> int:
        return int(self.prompt.shape[0])

    @property
    def n_arrivals(self) -> int:
        return int(sum(t[0].shape[0] for t in self.ticks))


def _lengths(seed: int, n: int, p_med, p_sig, p_lo, p_hi, d_med, d_sig, d_lo, d_hi, in_flight: bool):
    prompt = Stream(seed, 1).lognormal_int(n, p_med, p_sig, p_lo, p_hi)
    predicted = Stream(seed, 2).lognormal_int(n, d_med, d_sig, d_lo, d_hi)
    if in_flight:
        u = Stream(seed, 3).uniform(n)
        generated = np.minimum(np.floor(u * predicted).astype(np.int32), predicted - 1)
    else:
        generated = np.zeros(n, dtype=np.int32)
    return prompt, generated, predicted


# Real response lengths for the misprediction refinement.  The paper reports its length
# predictor's error on held-out data (Table 2: mean absolute error 78.25 tokens; 56.77 %,
# 68.79 % and 77.95 % of predictions within 25, 50 and 100 tokens).  The stand-in error is a
# two-component Laplace mixture with exactly that mean absolute error and about the same
# shares (53 %, 70 %, 81 %): most predictions close, a heavy tail of large misses.
ERR_WEIGHT, ERR_SCALE_NEAR, ERR_SCALE_FAR = 0.7, 20.0, 214.16666666666666   # 0.7*20 + 0.3*214.1667 = 78.25


def actual_lengths(seed: int, stream: int, predicted: np.ndarray, generated: np.ndarray | None = None) -> np.ndarray:
    """Real response length per request: predicted + error, at least 1 and, for a request that
    has already produced g tokens, at least g + 1 (it is still running)."""
    n = len(predicted)
    s = Stream(seed, stream)
    pick = s.uniform(n)
    u = s.uniform(n) - 0.5
    scale = np.where(pick < ERR_WEIGHT, ERR_SCALE_NEAR, ERR_SCALE_FAR)
    err = -scale * np.sign(u) * np.log(1.0 - 2.0 * np.abs(u))      # Laplace by inverse CDF
    act = np.rint(predicted.astype(np.float64) + err)
    lo = 1 if generated is None else generated.astype(np.float64) + 1
    return np.clip(np.maximum(act, lo), 1, 2 ** 30).astype(np.int32)


def make_actual(wl: "Workload", seed: int) -> Tuple[np.ndarray, List[np.ndarray]]:
    """Real lengths for a workload: one array for the in-flight table, one per tick of arrivals."""
    table = actual_lengths(seed, 6, wl.predicted, wl.generated)
    ticks = [actual_lengths(seed + 1000 + k, 6, ad) for k, (_, ad) in enumerate(wl.ticks)]
    return table, ticks


def _uniform_instances(seed: int, n: int, n_inst: int) -> np.ndarray:
    u = Stream(seed, 4).uniform(n)
    return np.minimum((u * n_inst).astype(np.int32), n_inst - 1)


def _zipf_instances(seed: int, n: int, n_inst: int, s: float) -> np.ndarray:
    """Instance k drawn with weight (k+1)^-s by inverting the cumulative weights."""
    w = np.arange(1, n_inst + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = Stream(seed, 4).uniform(n)
    return np.minimum(np.searchsorted(cdf, u, side="right"), n_inst - 1).astype(np.int32)


def _capacity(prompt, generated, instance, n_inst: int) -> int:
    """Capacity chosen so that the 80 % threshold sits at the median instance's present occupancy.

    The paper gives no token value for M (it is a property of the serving
    hardware).  A threshold at the median of the per-instance token counts
    (prompt + generated, summed per instance) keeps the memory-penalty term of
    the router active for about half of the instances under uniform and under
    Zipf assignment alike, so that the curves really decide routes.  M is a
    multiple of 5, so 0.8*M is a whole number of tokens.
    """
    tokens = prompt.astype(np.int64) + generated.astype(np.int64)
    per_inst = np.bincount(instance, weights=tokens.astype(np.float64), minlength=n_inst)
    med = int(np.median(per_inst)) if len(per_inst) else 0
    theta = max(4 * -(-med // 4), 4)
    return 5 * theta // 4


_SPECS = {
    # name, I, N, H, arrivals, zipf, (prompt median, sigma, lo, hi), (output median, sigma, lo, hi)
    0: ("tiny", 8, 256, 64, 32, None, (512, 1.0, 16, 4096), (256, 1.0, 1, 2048)),
    1: ("small", 64, 16384, 256, 1024, None, (512, 1.0, 16, 4096), (256, 1.0, 1, 2048)),
    2: ("medium", 512, 262144, 1024, 8192, 1.1, (1024, 1.2, 16, 8192), (384, 1.2, 1, 4096)),
    3: ("large", 4096, 2097152, 2048, 65536, None, (1024, 1.2, 16, 8192), (384, 1.2, 1, 4096)),
    4: ("streaming", 1024, 524288, 1024, None, None, (1024, 1.2, 16, 8192), (384, 1.2, 1, 4096)),
}

STREAM_TICKS = 1000
STREAM_MEAN = 4096
STREAM_BURST_EVERY = 100
STREAM_BURST_FACTOR = 4


def make_config(index: int, *, n_ticks: int | None = None, scale: float = 1.0) -> Workload:
    """Build configuration `index` (0..4).

    `n_ticks` shortens the streaming configuration (tests); `scale` shrinks the
    in-flight set and the arrival count of a one-shot configuration by a common
    factor while keeping instances, horizon and distributions (tests only).
    """
    name, n_inst, n_req, horizon, n_arr, zipf, pspec, dspec = _SPECS[index]
    seed = BASE_SEED + index
    n_req = max(1, int(round(n_req * scale)))
    prompt, generated, predicted = _lengths(seed, n_req, *pspec, *dspec, in_flight=True)
    if zipf is None:
        instance = _uniform_instances(seed, n_req, n_inst)
    else:
        instance = _zipf_instances(seed, n_req, n_inst, zipf)
    cap = _capacity(prompt, generated, instance, n_inst)

    ticks: List[Tuple[np.ndarray, np.ndarray]] = []
    if index != 4:
        n_arr = max(1, int(round(n_arr * scale)))
        ap, _, ad = _lengths(seed + 1000, n_arr, *pspec, *dspec, in_flight=False)
        ticks.append((ap, ad))
        streaming = False
    else:
        total_ticks = STREAM_TICKS if n_ticks is None else n_ticks
        counts = Stream(seed, 5)
        sizes = []
        for t in range(1, total_ticks + 1):
            lam = STREAM_MEAN * (STREAM_BURST_FACTOR if t % STREAM_BURST_EVERY == 0 else 1)
            sizes.append(counts.poisson(float(lam)))
        total = int(sum(sizes))
        ap, _, ad = _lengths(seed + 1000, total, *pspec, *dspec, in_flight=False)
        off = 0
        for s in sizes:
            ticks.append((ap[off:off + s].copy(), ad[off:off + s].copy()))
            off += s
        streaming = True

    wl = Workload(
        name=name, n_instances=n_inst, horizon=horizon,
        prompt=prompt, generated=generated, predicted=predicted, instance=instance,
        capacity_tokens=cap, ticks=ticks, streaming=streaming,
    )
    wl.max_requests = wl.n_requests + wl.n_arrivals
    return wl


def make_random(seed: int, n_inst: int, horizon: int, n_req: int, n_arr: int, *,
                max_prompt: int = 64, max_output: int = 48, capacity: int | None = None,
                t_mem: float = 0.8, beta: float = 1.0) -> Workload:
    """Small uniform-length workload for property tests (any I, H, N, A >= 0)."""
    s = Stream(seed, 9)
    prompt = (1 + (s.uniform(n_req) * max_prompt)).astype(np.int32)
    predicted = (1 + (s.uniform(n_req) * max_output)).astype(np.int32)
    generated = np.minimum((s.uniform(n_req) * predicted).astype(np.int32), predicted - 1)
    instance = np.minimum((s.uniform(n_req) * n_inst).astype(np.int32), n_inst - 1)
    ap = (1 + (s.uniform(n_arr) * max_prompt)).astype(np.int32)
    ad = (1 + (s.uniform(n_arr) * max_output)).astype(np.int32)
    cap = capacity if capacity is not None else _capacity(prompt, generated, instance, n_inst)
    wl = Workload(
        name=f"random{seed}", n_instances=n_inst, horizon=horizon,
        prompt=prompt, generated=generated, predicted=predicted, instance=instance,
        capacity_tokens=cap, t_mem=t_mem, beta=beta, ticks=[(ap, ad)],
    )
    wl.max_requests = n_req + n_arr
    return wl

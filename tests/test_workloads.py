import numpy as np
import pytest

from paper_2504_03702_b200 import workloads as W


def test_stream_is_counter_based_and_reproducible():
    a = W.Stream(7, 1).raw(10)
    s = W.Stream(7, 1)
    b = np.concatenate([s.raw(4), s.raw(6)])
    assert (a == b).all()
    assert (W.Stream(7, 2).raw(10) != a).any()
    u = W.Stream(1, 1).uniform(100000)
    assert 0.0 <= u.min() and u.max() < 1.0 and abs(u.mean() - 0.5) < 0.01
    z = W.Stream(1, 2).normal(200000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01


def test_poisson_mean():
    s = W.Stream(3, 5)
    draws = [s.poisson(4096.0) for _ in range(200)]
    assert abs(np.mean(draws) - 4096) < 4 * 64 / np.sqrt(200) + 1


@pytest.mark.parametrize("idx,n_inst,n_req,h,n_arr", [
    (0, 8, 256, 64, 32), (1, 64, 16384, 256, 1024), (2, 512, 262144, 1024, 8192)])
def test_config_shapes_and_ranges(idx, n_inst, n_req, h, n_arr):
    wl = W.make_config(idx)
    assert (wl.n_instances, wl.n_requests, wl.horizon, wl.n_arrivals) == (n_inst, n_req, h, n_arr)
    assert wl.prompt.dtype == np.int32 and wl.instance.dtype == np.int32
    assert wl.prompt.min() >= 16 and wl.predicted.min() >= 1
    assert (wl.generated >= 0).all() and (wl.generated < wl.predicted).all()
    assert wl.instance.min() >= 0 and wl.instance.max() < n_inst
    assert wl.capacity_tokens % 5 == 0
    ap, ad = wl.ticks[0]
    assert ap.min() >= 16 and ad.min() >= 1
    wl2 = W.make_config(idx)
    assert (wl2.prompt == wl.prompt).all() and (wl2.ticks[0][1] == ad).all()


def test_medians_follow_the_recipe():
    wl = W.make_config(2)
    assert abs(np.median(wl.prompt) - 1024) < 40
    assert abs(np.median(wl.predicted) - 384) < 20
    counts = np.bincount(wl.instance, minlength=512)
    assert counts[0] == counts.max() and counts[0] > 20 * counts[256:].mean()  # Zipf skew


def test_streaming_config_short():
    wl = W.make_config(4, n_ticks=100)
    assert wl.streaming and len(wl.ticks) == 100
    sizes = [len(t[0]) for t in wl.ticks]
    assert abs(np.mean(sizes[:99]) - 4096) < 40
    assert abs(sizes[99] - 4 * 4096) < 6 * 128
    assert wl.max_requests == wl.n_requests + sum(sizes)

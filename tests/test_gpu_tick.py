"""pre_tick: one scheduler tick (decode step, refinement, scaler signals) in one call.

Expected values are the oracle's three functions applied one after the other: orc_step (Sec. 2),
orc_refine (Sec. 4.3.1) and orc_scaler_signals (Sec. 4.3.2).  Everything is compared bit for bit.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2504_03702_b200 import binding as B  # noqa: E402
from paper_2504_03702_b200 import workloads as W  # noqa: E402
from paper_2504_03702_b200.state import DeviceState  # noqa: E402
from tests.gpu_util import assert_state_equal, dev  # noqa: E402


def both(wl):
    st = DeviceState.from_workload(wl)
    ref = oracle.State.from_workload(wl)
    st.anticipate()
    ref.anticipate()
    return st, ref


def one_tick(st, ref, actual_dev, actual_host, what, levels=(0.95, 0.10, 0.30)):
    counts, over, row_max, summary = st.tick(actual_dev, True, *levels)
    ref.step()
    want_counts = ref.refine(actual_host) if actual_host is not None else None
    w_over, w_max, w_sum = ref.scaler_signals(*levels)
    if want_counts is not None:
        assert counts.cpu().numpy().tolist() == want_counts.tolist(), f"event counts differ {what}"
    assert (over.cpu().numpy() == w_over).all(), f"cells above the level differ {what}"
    assert (row_max.cpu().numpy() == w_max).all(), f"row maxima differ {what}"
    assert summary.cpu().numpy().tolist() == w_sum.tolist(), f"summary differs {what}"
    return want_counts


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_tick_configs_after_a_routed_batch(idx):
    wl = W.make_config(idx)
    table_actual, tick_actual = W.make_actual(wl, W.BASE_SEED + idx)
    st, ref = both(wl)
    ap, ad = wl.ticks[0]
    st.route_batch(dev(ap), dev(ad), want_score=False)
    ref.route_batch(ap, ad, fast=True, want_score=False)
    actual = np.concatenate([table_actual, tick_actual[0]])
    actual_dev = dev(actual)
    events = np.zeros(3, np.int64)
    for t in range(24):
        # thresholds low enough that some rows count as overloaded and the sums are not trivial
        events += one_tick(st, ref, actual_dev, actual, f"tick {t}", levels=(0.5, 0.10, 0.9))
        if t % 6 == 5:
            assert_state_equal(st, ref, f"after tick {t}")
    assert_state_equal(st, ref, "at the end")
    assert events[0] > 0 and events[1] > 0 and events[2] == 0
    after = st.curves.clone()
    st.anticipate()                       # the maps still are what the build gives on the table
    assert (st.curves == after).all()
    assert st.status() == B.PRE_OK
    st.close()


@pytest.mark.parametrize("seed,n_inst,h,n", [(191, 1, 1, 5), (192, 3, 7, 70), (193, 9, 40, 1000), (194, 130, 33, 5000),
                                             (195, 2, 300, 64), (196, 5, 2048, 900), (197, 9000, 4, 30000)])
def test_tick_shapes_to_completion(seed, n_inst, h, n):
    wl = W.make_random(seed, n_inst, h, n, 0, max_prompt=50, max_output=40 if h < 1000 else 3000)
    err = np.rint((W.Stream(seed, 7).uniform(n) - 0.5) * 30).astype(np.int32)
    actual = np.maximum(1, wl.predicted + err).astype(np.int32)        # some real ends already lie behind
    actual_dev = dev(actual)
    st, ref = both(wl)
    for t in range(60 if h < 1000 else 12):
        one_tick(st, ref, actual_dev, actual, f"tick {t}", levels=(0.3, 0.05, 0.6))
    assert_state_equal(st, ref)
    st.close()


def test_tick_without_refinement_and_without_signals_equals_step():
    wl = W.make_config(1)
    st, ref = both(wl)
    for t in range(5):
        counts, over, row_max, summary = st.tick(None, False)
        assert counts is None and over is None and summary is None
        ref.step()
    assert_state_equal(st, ref, "plain ticks")
    for t in range(5):
        one_tick(st, ref, None, None, f"tick {t} with signals only")
    assert_state_equal(st, ref, "ticks with signals")
    assert st.status() == B.PRE_OK
    st.close()


def test_tick_streaming_ticks_with_arrivals():
    wl = W.make_config(4, n_ticks=10)
    table_actual, tick_actual = W.make_actual(wl, W.BASE_SEED + 4)
    st, ref = both(wl)
    actual = np.zeros(wl.max_requests, np.int32)
    actual[:wl.n_requests] = table_actual
    actual_dev = dev(actual)
    n = wl.n_requests
    for t, (ap, ad) in enumerate(wl.ticks):
        one_tick(st, ref, actual_dev, actual, f"tick {t}", levels=(0.6, 0.10, 0.9))
        c, _ = st.route_batch(dev(ap), dev(ad))
        wc, _ = ref.route_batch(ap, ad, fast=True)
        assert (c.cpu().numpy() == wc).all()
        actual[n:n + len(ap)] = tick_actual[t]
        actual_dev[n:n + len(ap)] = dev(tick_actual[t])
        n += len(ap)
    assert_state_equal(st, ref, "at the end of the stream")
    st.close()


def test_tick_malformed_rows_and_argument_errors():
    wl = W.make_random(198, 6, 32, 400, 0, max_prompt=60, max_output=50)
    actual = wl.predicted.copy()
    actual[7] = 0                      # no real length: malformed for the refinement only
    wl.instance[9] = 77                # malformed everywhere
    st, ref = both(wl)
    assert st.status() == B.PRE_EBADREQ
    for t in range(4):
        want = one_tick(st, ref, dev(actual), actual, f"tick {t}")
        assert want[2] == 2
        assert st.status() == B.PRE_EBADREQ
    assert_state_equal(st, ref)
    over = torch.zeros(6, dtype=torch.int32, device="cuda")
    code = B.pre_tick(st.ctx, st.prompt, st.generated, st.predicted, st.instance, None, st.n_requests, st.curves,
                      st.queued_p, st.current_d, 0.9, 0.1, 0.3, over, None, None, None)
    assert code == B.PRE_EINVAL
    st.close()

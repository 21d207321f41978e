"""Bounded device-side waits: what is left behind when one runs out.

Every wait in the kernels (the router's exchange between its blocks, the grid barriers and the
bulk-copy arrival of the fused anticipator build) gives up after a number of polls.  The test hook
pre_test_set_spin_limit sets that number to 0, so the first unsuccessful poll gives up: nothing
faults or hangs, the kernels leave through their ordinary give-up path.  These tests check the
status and the state the header promises after that, against the oracle.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2504_03702_b200 import binding as B  # noqa: E402
from paper_2504_03702_b200 import workloads as W  # noqa: E402
from paper_2504_03702_b200.state import DeviceState  # noqa: E402
from tests.gpu_util import assert_scores_close, assert_state_equal, dev  # noqa: E402


@pytest.mark.parametrize("idx", [1, 2])
def test_router_wait_that_runs_out_keeps_a_routed_prefix(idx):
    wl = W.make_config(idx)
    st = DeviceState.from_workload(wl)
    ref = oracle.State.from_workload(wl)
    st.anticipate()
    ref.anticipate()
    n0 = wl.n_requests
    ap, ad = wl.ticks[0]
    ap, ad = ap[:256], ad[:256]

    st.select_router(B.ROUTE_SCAN)      # the kernel whose blocks wait for one another
    assert B.pre_test_set_spin_limit(st.ctx, 0) == B.PRE_OK
    choice, score = st.route_batch(dev(ap), dev(ad))
    assert st.status() == B.PRE_ETIMEOUT
    routed = st.sync_count() - n0
    assert 0 <= routed < len(ap), "with no patience at all the batch cannot have been finished"
    got_c, got_s = choice.cpu().numpy(), score.cpu().numpy()
    want_c, want_s = ref.route_batch(ap[:routed], ad[:routed])
    assert (got_c[:routed] == want_c).all()
    assert_scores_close(got_s[:routed], want_s, got_c[:routed])
    assert (got_c[routed:] == -1).all() and (got_s[routed:] == 0.0).all()
    assert_state_equal(st, ref, "after the wait ran out")

    # the context is still good: the rest of the batch, with the usual patience
    assert B.pre_test_set_spin_limit(st.ctx, 1 << 22) == B.PRE_OK
    choice, score = st.route_batch(dev(ap[routed:]), dev(ad[routed:]))
    assert st.status() == B.PRE_OK
    want_c, want_s = ref.route_batch(ap[routed:], ad[routed:])
    assert (choice.cpu().numpy() == want_c).all()
    assert_scores_close(score.cpu().numpy(), want_s, want_c)
    assert_state_equal(st, ref, "after the rest of the batch")
    st.close()


def test_admission_router_wait_that_runs_out():
    wl = W.make_config(1)
    st = DeviceState.from_workload(wl)
    ref = oracle.State.from_workload(wl)
    st.anticipate()
    ref.anticipate()
    n0 = wl.n_requests
    ap, ad = wl.ticks[0]
    ap, ad = ap[:128], ad[:128]
    st.make_queue(16)
    st.select_router(B.ROUTE_SCAN)      # the kernel whose blocks wait for one another
    B.pre_test_set_spin_limit(st.ctx, 0)
    _, choice, score = st.route_admit(dev(ap), dev(ad), overload_level=0.95, overload_share=0.10)
    assert st.status() == B.PRE_ETIMEOUT
    routed = st.sync_count() - n0
    got_c = choice.cpu().numpy()
    want_c, _ = ref.route_batch(ap[:routed], ad[:routed])      # nothing blocks at these levels
    assert (got_c[:routed] == want_c).all() and (got_c[routed:] == -1).all()
    assert st.queue_state.cpu().tolist() == [0, 0]
    assert_state_equal(st, ref, "after the wait ran out")
    st.close()


def test_build_wait_that_runs_out_and_the_next_build():
    wl = W.make_config(2)
    st = DeviceState.from_workload(wl)
    ref = oracle.State.from_workload(wl)
    ref.anticipate()
    st.anticipate()                                   # a first build, so that the second one takes the quick layout
    assert st.status() == B.PRE_OK
    B.pre_test_set_spin_limit(st.ctx, 0)
    st.anticipate()                                   # the maps this leaves are undefined
    assert st.status() == B.PRE_ETIMEOUT
    B.pre_test_set_spin_limit(st.ctx, 1 << 22)
    for _ in range(2):                                # exact layout, then the learned one again
        st.curves.fill_(-1)
        st.anticipate()
        assert st.status() == B.PRE_OK
        assert (st.curves.cpu().numpy() == ref.curves).all()
        assert (st.current_d.cpu().numpy() == ref.current_d).all()
    st.close()

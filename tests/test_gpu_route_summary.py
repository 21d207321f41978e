"""The routing kernel that works on per-row summaries, on the inputs that take its special paths.

Every case is compared with the oracle's literal router decision by decision; the cases are built
so that a particular path of the kernel is certain to run: rows whose summary only bounds the peak
(scanned cell by cell), the same row winning several arrivals in a row (a decision has to wait for
a fold), whole-number and binary64 scores, every fold-thread layout, and the hand-over to the
scanning kernel when a value could leave 32 bits or the instances do not fit shared memory.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_03702_b200 import workloads as W

pytestmark = pytest.mark.gpu

from gpu_util import assert_scores_close, assert_state_equal, dev  # noqa: E402
from paper_2504_03702_b200 import binding as B  # noqa: E402
from paper_2504_03702_b200.state import DeviceState  # noqa: E402


def route_and_compare(wl, ap, ad, path=B.ROUTE_SUMMARY, batches=1):
    st = DeviceState.from_workload(wl)
    if path is not None:
        st.select_router(path)
    ref = oracle.State.from_workload(wl)
    st.anticipate()
    ref.anticipate()
    cuts = np.linspace(0, len(ap), batches + 1).astype(int)
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        choice, score = st.route_batch(dev(ap[lo:hi]), dev(ad[lo:hi]))
        want_c, want_s = ref.route_batch(ap[lo:hi], ad[lo:hi])
        got = choice.cpu().numpy()
        assert (got == want_c).all(), f"first difference at arrival {lo + int(np.argmax(got != want_c))}"
        assert_scores_close(score.cpu().numpy(), want_s, want_c)
    assert_state_equal(st, ref)
    assert st.status() == B.PRE_OK
    st.close()
    return ref


def rising_maps(seed, n_inst, h, n, beta=1.0, capacity=None):
    """Requests with short prompts that all outlast the window: every map rises with the step, the
    largest cell + step sits at the last step, and no arrival's ramp reaches it."""
    wl = W.make_random(seed, n_inst, h, n, 0, max_prompt=4, max_output=8, capacity=capacity, beta=beta)
    wl.predicted[:] = 3 * h + 5
    wl.generated[:] = np.arange(n, dtype=np.int32) % 7
    return wl


@pytest.mark.parametrize("beta,t_mem", [(1.0, 0.8), (2.0, 0.8), (0.75, 0.8), (1.0, 0.81237)])
def test_rows_that_are_only_bounded_are_scanned(beta, t_mem):
    wl = rising_maps(51, 37, 96, 900, beta=beta, capacity=40000)
    wl.t_mem = t_mem
    rng = np.random.default_rng(5)
    ap = rng.integers(0, 3000, 300).astype(np.int32)
    ad = rng.integers(1, 96, 300).astype(np.int32)      # every ramp ends before the last step
    wl.max_requests = 900 + 300
    before = oracle.State.from_workload(wl)
    before.anticipate()
    top = before.curves + np.arange(96)[None, :]
    assert (top.argmax(axis=1) == 95).all(), "the maps were meant to peak at the end of the window"
    route_and_compare(wl, ap, ad)


@pytest.mark.parametrize("beta", [1.0, 0.5])
def test_bounded_and_exact_rows_mixed(beta):
    """Half of the instances hold rising maps, the other half ordinary ones; short and long arrivals."""
    a = rising_maps(52, 20, 64, 400, beta=beta, capacity=30000)
    b = W.make_random(53, 20, 64, 400, 0, max_prompt=200, max_output=150, capacity=30000, beta=beta)
    wl = a
    wl.prompt = np.concatenate([a.prompt, b.prompt])
    wl.generated = np.concatenate([a.generated, b.generated])
    wl.predicted = np.concatenate([a.predicted, b.predicted])
    wl.instance = np.concatenate([a.instance, b.instance + 20]).astype(np.int32)
    wl.n_instances = 40
    rng = np.random.default_rng(6)
    ap = rng.integers(0, 500, 400).astype(np.int32)
    ad = np.where(rng.random(400) < 0.5, rng.integers(1, 4, 400), rng.integers(1, 300, 400)).astype(np.int32)
    wl.max_requests = 800 + 400
    route_and_compare(wl, ap, ad, batches=3)


@pytest.mark.parametrize("n_inst", [1, 2, 3, 5])
@pytest.mark.parametrize("beta", [1.0, 0.3])
def test_the_same_rows_win_again_and_again(n_inst, beta):
    """Few instances: a row that has just received an arrival is often the best one for the next."""
    wl = W.make_random(60 + n_inst, n_inst, 48, 60, 0, max_prompt=50, max_output=90, beta=beta)
    rng = np.random.default_rng(7)
    ap = rng.integers(0, 40, 500).astype(np.int32)
    ad = rng.integers(1, 120, 500).astype(np.int32)
    wl.max_requests = 60 + 500
    route_and_compare(wl, ap, ad, batches=2)


def test_one_almost_empty_instance_takes_a_long_run_of_arrivals():
    wl = W.make_random(70, 12, 80, 3000, 0, max_prompt=400, max_output=200)
    keep = wl.instance != 4
    keep[:3] = True
    for name in ("prompt", "generated", "predicted", "instance"):
        setattr(wl, name, getattr(wl, name)[keep])
    rng = np.random.default_rng(8)
    ap = rng.integers(1, 30, 600).astype(np.int32)
    ad = rng.integers(1, 60, 600).astype(np.int32)
    wl.max_requests = len(wl.prompt) + 600
    ref = route_and_compare(wl, ap, ad)
    assert (ref.instance[len(wl.prompt):len(wl.prompt) + 50] == 4).mean() > 0.5


@pytest.mark.parametrize("h", [1, 2, 7, 255, 1024, 1025, 2048, 2050, 4096, 4099, 8192])
def test_every_fold_layout(h):
    """Horizons on both sides of each cells-per-thread step, even and odd."""
    wl = W.make_random(80 + h % 50, 9, h, 150, 0, max_prompt=300, max_output=2 * h + 5)
    rng = np.random.default_rng(9)
    ap = rng.integers(0, 300, 120).astype(np.int32)
    ad = rng.integers(1, 2 * h + 5, 120).astype(np.int32)
    wl.max_requests = 150 + 120
    route_and_compare(wl, ap, ad)


def test_malformed_arrivals_and_a_full_table_on_the_summary_kernel():
    wl = W.make_random(90, 30, 32, 400, 0)
    rng = np.random.default_rng(10)
    ap = rng.integers(0, 60, 200).astype(np.int32)
    ad = rng.integers(1, 50, 200).astype(np.int32)
    ad[[0, 33, 64, 65, 199]] = 0
    ap[[31, 32, 100]] = -1
    wl.max_requests = 400 + 170
    st = DeviceState.from_workload(wl)
    st.select_router(B.ROUTE_SUMMARY)
    ref = oracle.State.from_workload(wl)
    st.anticipate()
    ref.anticipate()
    choice, score = st.route_batch(dev(ap), dev(ad))
    want_c, want_s = ref.route_batch(ap, ad)
    assert (choice.cpu().numpy() == want_c).all()
    assert_scores_close(score.cpu().numpy(), want_s, want_c)
    assert (score.cpu().numpy()[want_c < 0] == 0.0).all()
    assert_state_equal(st, ref)
    assert st.status() == B.PRE_ECAPACITY
    choice, _ = st.route_batch(dev(ap[:5]), dev(ad[:5]))          # the table is full now
    assert (choice.cpu().numpy() == -1).all()
    st.close()


def test_values_that_could_leave_32_bits_go_to_the_scanning_kernel():
    """The summary kernel declines the batch on the device; the result is the scanning kernel's."""
    wl = W.make_random(91, 25, 40, 3000, 0, max_prompt=2 ** 22, max_output=60, capacity=10 ** 9)
    rng = np.random.default_rng(11)
    ap = rng.integers(2 ** 26, 2 ** 27, 80).astype(np.int32)       # 80 such prompts can add 2^33 to a cell
    ad = rng.integers(1, 80, 80).astype(np.int32)
    wl.max_requests = 3000 + 80
    route_and_compare(wl, ap, ad)
    wl = W.make_random(92, 25, 40, 3000, 0, max_prompt=2 ** 27, max_output=60, capacity=10 ** 11)   # cells above 2^32 already
    wl.max_requests = 3000 + 80
    route_and_compare(wl, (ap // 1000).astype(np.int32), ad)


def test_whole_number_scores_that_could_reach_2_to_the_30_go_to_the_scanning_kernel():
    """beta and theta are whole numbers, so the context gets the whole-number kind of the summary kernel; with
    beta = 4096 and peaks around 2^19 the score bound passes 2^30 and the kernel declines on the device."""
    wl = W.make_random(97, 25, 40, 600, 0, max_prompt=2 ** 16, max_output=60, capacity=10 ** 5, beta=4096.0)
    rng = np.random.default_rng(15)
    ap = rng.integers(2 ** 12, 2 ** 14, 120).astype(np.int32)
    ad = rng.integers(1, 80, 120).astype(np.int32)
    wl.max_requests = 600 + 120
    ref = route_and_compare(wl, ap, ad)
    assert ref.curves.max() * 4096.0 > 2.0 ** 30, "the case was meant to pass the whole-number bound"


def test_selecting_the_kernel():
    wl = W.make_random(93, 20000, 4, 100, 0)
    st = DeviceState.from_workload(wl)
    assert B.pre_route_select(st.ctx, B.ROUTE_SUMMARY) == B.PRE_ESIZE       # too many instances for one block
    assert B.pre_route_select(st.ctx, 3) == B.PRE_EINVAL
    assert B.pre_route_select(st.ctx, -1) == B.PRE_EINVAL
    assert B.pre_route_select(st.ctx, B.ROUTE_SCAN) == B.PRE_OK
    assert B.pre_route_select(st.ctx, B.ROUTE_AUTO) == B.PRE_OK
    assert B.pre_route_select(None, B.ROUTE_AUTO) == B.PRE_EINVAL
    st.close()
    wl = W.make_random(94, 300, 16, 2000, 0)
    rng = np.random.default_rng(12)
    ap = rng.integers(0, 100, 300).astype(np.int32)
    ad = rng.integers(1, 40, 300).astype(np.int32)
    wl.max_requests = 2300
    for path in (B.ROUTE_AUTO, B.ROUTE_SCAN, B.ROUTE_SUMMARY):
        route_and_compare(wl, ap, ad, path=path)


def test_many_instances_with_binary64_scores_take_the_scanning_kernel():
    """More than 5,120 instances give a score lane more rows than the binary64 kind of the summary kernel
    keeps in registers: selecting that kernel outright is refused, the default routes with the other."""
    wl = W.make_random(96, 6000, 8, 20000, 0, max_prompt=100, max_output=20, beta=0.75)
    st = DeviceState.from_workload(wl)
    assert B.pre_route_select(st.ctx, B.ROUTE_SUMMARY) == B.PRE_ESIZE
    st.close()
    rng = np.random.default_rng(14)
    ap = rng.integers(0, 100, 200).astype(np.int32)
    ad = rng.integers(1, 20, 200).astype(np.int32)
    wl.max_requests = 20200
    route_and_compare(wl, ap, ad, path=B.ROUTE_AUTO)
    wl.beta = 2.0      # whole-number scores: the summary kernel takes this many instances
    route_and_compare(wl, ap, ad, path=B.ROUTE_SUMMARY)


def test_many_instances_close_to_the_shared_memory_limit():
    wl = W.make_random(95, 9300, 8, 30000, 0, max_prompt=100, max_output=20)
    rng = np.random.default_rng(13)
    ap = rng.integers(0, 100, 400).astype(np.int32)
    ad = rng.integers(1, 20, 400).astype(np.int32)
    wl.max_requests = 30400
    route_and_compare(wl, ap, ad)


@pytest.mark.parametrize("n_inst", [40, 700, 2100])
@pytest.mark.parametrize("path", [B.ROUTE_SUMMARY, B.ROUTE_SCAN])
def test_equal_scores_go_to_the_lowest_index(n_inst, path):
    """Empty instances and identical arrivals: every score is shared by many rows, in the same lane, in
    other lanes of the warp and in other warps, and the lowest index among them has to win each time
    (Sec. 4.3.3 names no tie rule; the oracle's argmin takes the first)."""
    wl = W.make_random(3, n_inst, 64, 0, 0, capacity=100000)
    n = 3 * n_inst + 17
    ap = np.full(n, 10, dtype=np.int32)
    ad = np.full(n, 5, dtype=np.int32)
    wl.max_requests = n
    ref = route_and_compare(wl, ap, ad, path=path)
    assert ref.instance[:n].tolist() == [k % n_inst for k in range(n)]


def test_streaming_ticks_on_both_kernels():
    """Route, step, route ... over the first ticks of the streaming configuration, both kernels in turn."""
    wl = W.make_config(4, n_ticks=4)
    st = DeviceState.from_workload(wl)
    ref = oracle.State.from_workload(wl)
    st.anticipate()
    ref.anticipate()
    for t, (ap, ad) in enumerate(wl.ticks):
        st.select_router(B.ROUTE_SUMMARY if t % 2 == 0 else B.ROUTE_SCAN)
        st.step()
        ref.step()
        choice, score = st.route_batch(dev(ap), dev(ad))
        want_c, want_s = ref.route_batch(ap, ad, fast=True)
        assert (choice.cpu().numpy() == want_c).all(), f"tick {t}"
        assert_scores_close(score.cpu().numpy(), want_s, want_c)
    assert_state_equal(st, ref)
    st.close()


@pytest.mark.parametrize("beta,level", [(1.0, 0.7), (0.75, 0.7), (0.4, 0.5)])
def test_admission_queue_on_the_summary_kernel(beta, level):
    """Several calls with a queue that fills and drains, whole-number and binary64 scores, the kernel selected outright."""
    wl = W.make_random(96, 5, 24, 120, 0, max_prompt=200, max_output=60, beta=beta)
    wl.max_requests = 120 + 400
    st = DeviceState.from_workload(wl)
    st.select_router(B.ROUTE_SUMMARY)
    ref = oracle.State.from_workload(wl)
    st.anticipate()
    ref.anticipate()
    st.make_queue(12)
    ref.make_queue(12)
    rng = np.random.default_rng(14)
    seen = set()
    for call in range(10):
        a = int(rng.integers(0, 40))
        ap = rng.integers(0, 200, a).astype(np.int32)
        ad = rng.integers(1, 60, a).astype(np.int32)
        if a > 3 and call % 3 == 1:
            ad[1] = 0                                   # malformed
        waiting = int(ref.queue_state[1])
        qc, c, s = st.route_admit(dev(ap), dev(ad), overload_level=level, overload_share=0.10)
        wqc, wc, ws = ref.route_admit(ap, ad, overload_level=level, overload_share=0.10)
        assert (c.cpu().numpy() == wc).all(), f"call {call}: arrivals"
        assert (qc[:waiting].cpu().numpy() == wqc).all(), f"call {call}: waiting requests"
        assert_scores_close(s.cpu().numpy(), ws, wc)
        assert st.queue_state.cpu().tolist() == ref.queue_state.tolist()
        assert_state_equal(st, ref, f"after call {call}")
        seen.update(np.unique(wc).tolist())
        seen.update((-10 - v for v in np.unique(wqc).tolist() if v >= 0))
        st.status()
        for _ in range(int(rng.integers(0, 4))):
            st.step()
            ref.step()
    assert -2 in seen and -3 in seen and any(v >= 0 for v in seen) and any(v <= -10 for v in seen), \
        "the case was meant to route, queue, turn away and route out of the queue"
    st.close()

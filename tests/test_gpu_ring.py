"""Full-width maps kept as a ring (pre_ring_step, pre_ring_window, pre_ring_fold) against the
oracle's router on full-width maps, tick by tick, through the C-ABI.

The device keeps ring[I][L] and routes on the window of width l; the oracle keeps the dense
maps of width L, takes peaks over their first l steps and shifts them on every step.  Bar: ring
(read out in logical order), backlog words, table and decisions bit-exact, scores within 1e-12.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_03702_b200 import workloads as W

pytestmark = pytest.mark.gpu

from gpu_util import assert_scores_close, dev, table  # noqa: E402
from paper_2504_03702_b200 import binding as B  # noqa: E402
from paper_2504_03702_b200.state import DeviceState  # noqa: E402


def pair(wl, width, window, extra_rows):
    """Device state whose own maps are the window, with a ring of `width`; oracle state of `width`."""
    cap = wl.n_requests + extra_rows
    st = DeviceState(wl.n_instances, window, wl.capacity_tokens, max(cap, 1), wl.t_mem, wl.beta)
    st.load_requests(wl.prompt, wl.generated, wl.predicted, wl.instance)
    st.make_ring(width)
    ref = oracle.State(wl.n_instances, width, wl.capacity_tokens, wl.prompt, wl.generated, wl.predicted,
                       wl.instance, max(cap, 1), wl.t_mem, wl.beta)
    ref.anticipate()
    return st, ref


def same(st, ref, what):
    assert (st.ring_logical().cpu().numpy() == ref.curves).all(), f"ring differs {what}"
    assert (st.current_d.cpu().numpy() == ref.current_d).all(), f"current_d differs {what}"
    assert (st.queued_p.cpu().numpy() == ref.queued_p).all(), f"queued_p differs {what}"
    n = st.sync_count()
    assert n == int(ref.n[0])
    for got, want in zip(table(st), (ref.prompt, ref.generated, ref.predicted, ref.instance)):
        assert (got == want[:n]).all(), f"table differs {what}"


def tick(st, ref, ap, ad, window):
    st.ring_step()
    ref.step()
    st.ring_window()
    choice, score = st.route_batch(dev(ap), dev(ad))
    st.ring_fold(dev(ap), dev(ad), choice)
    want_c, want_s = ref.route_window(ap, ad, window)
    assert (choice.cpu().numpy() == want_c).all()
    assert_scores_close(score.cpu().numpy(), want_s, want_c)


@pytest.mark.parametrize("seed,n_inst,width,window,n,a,ticks", [
    (71, 1, 5, 2, 12, 4, 14),          # the head goes round the ring several times
    (72, 6, 40, 7, 150, 20, 50),
    (73, 37, 96, 96, 600, 33, 12),     # window = width
    (74, 300, 257, 100, 4000, 150, 6),
    (75, 9, 16, 1, 80, 10, 20),
])
def test_ring_ticks_match_the_oracle(seed, n_inst, width, window, n, a, ticks):
    # responses up to twice the width: some requests reach beyond the map and enter it later
    wl = W.make_random(seed, n_inst, width, n, 0, max_prompt=300, max_output=2 * width)
    st, ref = pair(wl, width, window, a * ticks)
    same(st, ref, "after the build")
    rng = np.random.RandomState(seed)
    for t in range(ticks):
        ap = rng.randint(1, 300, a).astype(np.int32)
        ad = rng.randint(1, 2 * width + 1, a).astype(np.int32)
        if t == 1 and a > 3:
            ap[2] = -5                                 # malformed: dropped, result -1
        tick(st, ref, ap, ad, window)
        same(st, ref, f"after tick {t}")
    assert st.status() in (B.PRE_OK, B.PRE_EBADREQ)
    # the ring still is what the definition gives for the table as it stands
    n_rows = st.sync_count()
    check = oracle.State(n_inst, width, wl.capacity_tokens, ref.prompt[:n_rows], ref.generated[:n_rows],
                         ref.predicted[:n_rows], ref.instance[:n_rows], n_rows)
    check.anticipate()
    assert (st.ring_logical().cpu().numpy() == check.curves).all()
    st.close()


@pytest.mark.parametrize("seed,n_inst,width,window,n,a,ticks", [(77, 5, 24, 6, 120, 12, 60), (78, 40, 130, 100, 900, 40, 30)])
def test_ring_ticks_with_refinement_match_the_oracle(seed, n_inst, width, window, n, a, ticks):
    """A tick with the correction against real lengths: step, refine, window, route, fold."""
    wl = W.make_random(seed, n_inst, width, n, 0, max_prompt=200, max_output=width)
    st, ref = pair(wl, width, window, a * ticks)
    rng = np.random.RandomState(seed)
    cap = n + a * ticks
    actual = np.ones(cap, np.int32)
    actual[:n] = np.maximum(wl.generated + 1, wl.predicted + rng.randint(-15, 16, n)).astype(np.int32)
    actual_dev = dev(actual)
    early = extended = 0
    for t in range(ticks):
        ap = rng.randint(1, 200, a).astype(np.int32)
        ad = rng.randint(1, width + 1, a).astype(np.int32)
        n_before = int(ref.n[0])
        actual[n_before:n_before + a] = np.maximum(1, ad + rng.randint(-15, 16, a))
        actual_dev[n_before:n_before + a] = dev(actual[n_before:n_before + a])
        st.ring_step()
        ref.step()
        got = st.ring_refine(actual_dev).cpu().numpy()
        want = ref.refine(actual)
        assert (got == want).all(), f"refinement counts differ at tick {t}"
        early += int(want[0]); extended += int(want[1])
        st.ring_window()
        choice, score = st.route_batch(dev(ap), dev(ad))
        st.ring_fold(dev(ap), dev(ad), choice)
        want_c, want_s = ref.route_window(ap, ad, window)
        assert (choice.cpu().numpy() == want_c).all()
        assert_scores_close(score.cpu().numpy(), want_s, want_c)
        same(st, ref, f"after tick {t}")
    assert early > 0 and extended > 0
    assert st.status() == B.PRE_OK
    st.close()


@pytest.mark.parametrize("level", [0.7, 0.8])
def test_ring_ticks_with_the_admission_queue(level):
    """Full-width maps with pre_route_admit: waiting requests are routed out of the queue while arrivals
    join it, and the ring is brought up to date from the rows the call appended to the request table.
    The oracle routes on the first `window` steps of its full-width maps (its admission router on a state
    of that width) and rebuilds the full-width maps from the table by the definition."""
    seed, n_inst, width, window, n, a, ticks, qcap = 79, 6, 48, 10, 300, 24, 14, 40
    wl = W.make_random(seed, n_inst, width, n, 0, max_prompt=300, max_output=2 * width)
    cap = wl.n_requests + a * ticks + qcap
    st = DeviceState(n_inst, window, wl.capacity_tokens, cap, wl.t_mem, wl.beta)
    st.load_requests(wl.prompt, wl.generated, wl.predicted, wl.instance)
    st.make_ring(width)
    st.make_queue(qcap)
    full = oracle.State(n_inst, width, wl.capacity_tokens, wl.prompt, wl.generated, wl.predicted, wl.instance,
                        cap, wl.t_mem, wl.beta)
    full.anticipate()
    queue = None
    rng = np.random.RandomState(seed)
    routed_from_queue = joined = turned_away = 0
    for t in range(ticks):
        ap = rng.randint(1, 300, a).astype(np.int32)
        ad = rng.randint(1, 2 * width + 1, a).astype(np.int32)
        st.ring_step()
        full.step()
        st.ring_window()
        nf = int(full.n[0])
        win = oracle.State(n_inst, window, wl.capacity_tokens, full.prompt[:nf], full.generated[:nf],
                           full.predicted[:nf], full.instance[:nf], cap, wl.t_mem, wl.beta)
        win.curves[:] = full.curves[:, :window]
        win.queued_p[:] = full.queued_p
        win.current_d[:] = full.current_d
        win.make_queue(qcap)
        if queue is not None:
            win.queue_prompt[:], win.queue_predicted[:], win.queue_state[:] = queue
        waiting = int(win.queue_state[1])
        n0 = st.sync_count()
        qc, c, sc = st.route_admit(dev(ap), dev(ad), overload_level=level, overload_share=0.10)
        n1 = st.sync_count()
        if n1 > n0:   # the routed requests, each with its instance: the rows the call appended
            st.ring_fold(st.prompt[n0:n1], st.predicted[n0:n1], st.instance[n0:n1])
        want_qc, want_c, want_s = win.route_admit(ap, ad, level, 0.10)
        queue = (win.queue_prompt.copy(), win.queue_predicted.copy(), win.queue_state.copy())
        assert (qc.cpu().numpy()[:waiting] == want_qc).all(), f"tick {t}: waiting requests"
        assert (c.cpu().numpy() == want_c).all(), f"tick {t}: arrivals"
        assert_scores_close(sc.cpu().numpy(), want_s, want_c)
        assert st.queue_state.cpu().tolist() == win.queue_state.tolist()
        routed_from_queue += int((want_qc >= 0).sum())
        joined += int((want_c == -2).sum())
        turned_away += int((want_c == -3).sum())
        nf = int(win.n[0])
        full = oracle.State(n_inst, width, wl.capacity_tokens, win.prompt[:nf], win.generated[:nf],
                            win.predicted[:nf], win.instance[:nf], cap, wl.t_mem, wl.beta)
        full.anticipate()
        full.queued_p[:] = win.queued_p
        same(st, full, f"after tick {t}")
    assert routed_from_queue > 0 and joined > 0 and turned_away > 0, "the case was meant to exercise the queue"
    st.close()


def test_ring_streaming_config_first_ticks():
    """The streaming configuration on maps of its full width (1,024) with the paper's window of 100."""
    wl = W.make_config(4, n_ticks=3)
    st, ref = pair(wl, wl.horizon, 100, sum(len(t[0]) for t in wl.ticks))
    for t, (ap, ad) in enumerate(wl.ticks):
        tick(st, ref, ap, ad, 100)
        same(st, ref, f"after tick {t}")
    assert st.status() == B.PRE_OK
    st.close()


def test_ring_argument_errors_launch_nothing():
    wl = W.make_random(76, 4, 16, 10, 0)
    st, _ = pair(wl, 16, 8, 4)
    assert B.pre_ring_window(st.ctx, st.ring, 7, st.head, st.curves) == B.PRE_EINVAL      # narrower than the window
    assert B.pre_ring_window(st.ctx, None, 16, st.head, st.curves) == B.PRE_EINVAL
    assert B.pre_ring_fold(st.ctx, None, None, None, 3, st.ring, 16, st.head) == B.PRE_EINVAL
    assert B.pre_ring_fold(st.ctx, None, None, None, 0, st.ring, 16, st.head) == B.PRE_OK  # an empty batch
    assert B.pre_ring_step(st.ctx, st.prompt, st.generated, st.predicted, st.instance, st.n_requests, st.ring, 16,
                           None, st.queued_p, st.current_d) == B.PRE_EINVAL
    torch.cuda.synchronize()
    st.close()

"""CUDA path against the CPU oracle, element by element, through the C-ABI.

Bar: int64 curves, counters, table columns and routing decisions bit-exact; the binary64
score within 1e-12 relative (in practice identical: both sides round every operation
separately).
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


def both(wl):
    st = DeviceState.from_workload(wl)
    ref = oracle.State.from_workload(wl)
    st.anticipate()
    ref.anticipate()
    return st, ref


# ------------------------------------------------------------------ anticipator

@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_anticipate_configs(idx):
    wl = W.make_config(idx)
    st, ref = both(wl)
    assert_state_equal(st, ref, f"config {idx}")
    assert st.status() == B.PRE_OK
    # integer atomics commute: a second build gives the same bits
    first = st.curves.clone()
    st.anticipate()
    assert torch.equal(first, st.curves)
    st.close()


SHAPES = [(1, 1, 1, 7), (2, 3, 5, 0), (3, 1, 33, 50), (4, 7, 1, 90), (5, 5, 63, 400), (6, 9, 130, 700),
          (7, 300, 6, 5000), (8, 2, 4097, 300), (9, 1, 8192, 100), (10, 1200, 10, 20000), (11, 37, 250, 3000)]


@pytest.mark.parametrize("seed,n_inst,h,n", SHAPES)
def test_anticipate_shapes(seed, n_inst, h, n):
    wl = W.make_random(seed, n_inst, h, n, 0, max_prompt=500, max_output=3 * h + 5)
    st, ref = both(wl)
    assert_state_equal(st, ref)
    assert st.status() == B.PRE_OK
    st.close()


def test_anticipate_more_tiles_than_a_block_can_count():
    """8,300 one-row tiles: the build takes its slow path (global per-tile cursors)."""
    wl = W.make_random(16, 8300, 4096, 20000, 0, max_prompt=3000, max_output=6000)
    st, ref = both(wl)
    assert_state_equal(st, ref)
    st.anticipate()
    assert (st.curves.cpu().numpy() == ref.curves).all()
    assert st.status() == B.PRE_OK
    st.close()


def test_anticipate_all_on_one_instance_and_long_requests():
    wl = W.make_random(12, 6, 64, 3000, 0, max_prompt=4000, max_output=900)
    wl.instance[:] = 4
    st, ref = both(wl)
    assert_state_equal(st, ref)
    st.close()


def test_anticipate_sums_beyond_32_bits():
    """Prompts near the field limit: a tile's sum of B passes 2^32, so the build works in 64 bits."""
    wl = W.make_random(19, 3, 40, 500, 0, max_prompt=2 ** 27, max_output=90)
    st, ref = both(wl)
    assert int(ref.curves.max()) > 2 ** 32
    assert_state_equal(st, ref)
    wl = W.make_random(20, 70, 2048, 4000, 0, max_prompt=2 ** 27, max_output=5000)
    wl.instance[:] = wl.instance % 3 + 66           # a ragged last tile, all of it wide
    st2, ref2 = both(wl)
    assert_state_equal(st2, ref2)
    assert st.status() == B.PRE_OK and st2.status() == B.PRE_OK
    st.close()
    st2.close()


def test_anticipate_table_ordered_by_instance():
    """A table kept in instance order: every chunk holds long pieces of a few tiles."""
    wl = W.make_random(21, 64, 256, 60000, 0, max_prompt=3000, max_output=700)
    order = np.argsort(wl.instance, kind="stable")
    for name in ("prompt", "generated", "predicted", "instance"):
        setattr(wl, name, np.ascontiguousarray(getattr(wl, name)[order]))
    st, ref = both(wl)
    assert_state_equal(st, ref)
    st.close()


def test_anticipate_more_chunks_than_a_tile_block_has_threads():
    """300,000 requests are cut into 293 chunks while a tile block of this shape has 256 threads:
    a thread gathers from more than one chunk per tile (only its first is looked ahead)."""
    wl = W.make_random(22, 600, 1024, 300000, 0, max_prompt=2000, max_output=1500)
    st, ref = both(wl)
    assert_state_equal(st, ref)
    assert st.status() == B.PRE_OK
    st.close()


def test_anticipate_tombstones_and_malformed():
    wl = W.make_random(13, 5, 40, 600, 0)
    wl.generated[::7] = wl.predicted[::7]          # finished: silently ignored
    wl.generated[5] = wl.predicted[5] + 3
    st, ref = both(wl)
    assert_state_equal(st, ref)
    assert st.status() == B.PRE_OK
    st.close()
    wl.instance[11] = 5                             # out of range
    wl.instance[12] = -1
    wl.predicted[13] = 0
    wl.generated[14] = -2
    wl.prompt[15] = -1
    wl.prompt[16] = 2 ** 28                         # above the documented field limit
    st, ref = both(wl)
    ref2 = oracle.State.from_workload(wl)
    ref2.predicted[16] = 0                          # the oracle has no field limit: drop that one
    ref2.anticipate()
    assert (st.curves.cpu().numpy() == ref2.curves).all()
    assert (st.current_d.cpu().numpy() == ref2.current_d).all()
    assert st.status() == B.PRE_EBADREQ
    assert st.status() == B.PRE_OK                  # reading clears
    st.close()


def test_anticipate_prefix_of_table():
    wl = W.make_random(14, 8, 32, 1000, 0)
    st = DeviceState.from_workload(wl)
    st.anticipate(n_requests=400)
    ref = oracle.State(8, 32, wl.capacity_tokens, wl.prompt[:400], wl.generated[:400], wl.predicted[:400],
                       wl.instance[:400], 400)
    ref.anticipate()
    assert (st.curves.cpu().numpy() == ref.curves).all()
    st.anticipate(n_requests=0)
    assert int(st.curves.abs().sum()) == 0 and int(st.current_d.abs().sum()) == 0
    st.close()


def test_two_contexts_of_different_shapes():
    """Kernel attributes are process-wide: a second, smaller context must not break the first."""
    big = W.make_random(17, 64, 2048, 3000, 50, max_output=3000)
    small = W.make_random(18, 5, 64, 200, 20)
    st_big, ref_big = both(big)
    st_small, ref_small = both(small)
    st_big.anticipate()
    c, _ = st_big.route_batch(dev(big.ticks[0][0]), dev(big.ticks[0][1]))
    assert (c.cpu().numpy() == ref_big.route_batch(*big.ticks[0])[0]).all()
    c, _ = st_small.route_batch(dev(small.ticks[0][0]), dev(small.ticks[0][1]))
    assert (c.cpu().numpy() == ref_small.route_batch(*small.ticks[0])[0]).all()
    assert_state_equal(st_big, ref_big)
    assert_state_equal(st_small, ref_small)
    st_big.close()
    st_small.close()


def test_argument_errors_launch_nothing():
    wl = W.make_random(15, 4, 16, 10, 0)
    st = DeviceState.from_workload(wl)
    assert B.pre_anticipate(st.ctx, st.prompt, st.generated, st.predicted, st.instance, -1, st.curves,
                            st.current_d) == B.PRE_EINVAL
    assert B.pre_anticipate(st.ctx, st.prompt, st.generated, st.predicted, st.instance, 10 ** 6, st.curves,
                            st.current_d) == B.PRE_EINVAL
    assert B.pre_anticipate(st.ctx, st.prompt, st.generated, st.predicted, st.instance, 10, None,
                            st.current_d) == B.PRE_EINVAL
    assert B.pre_anticipate(st.ctx, st.prompt, st.generated, st.predicted, st.instance, 10,
                            st.curves.data_ptr() + 8, st.current_d) == B.PRE_EINVAL   # misaligned
    assert B.pre_anticipate(st.ctx, None, st.generated, st.predicted, st.instance, 10, st.curves,
                            st.current_d) == B.PRE_EINVAL
    assert st.status() == B.PRE_OK
    st.close()


# ------------------------------------------------------------------ router

@pytest.mark.parametrize("idx", [0, 1, 2])
def test_route_configs_against_literal_oracle(idx, router):
    wl = W.make_config(idx)
    st, ref = both(wl)
    ap, ad = wl.ticks[0]
    choice, score = st.route_batch(dev(ap), dev(ad))
    want_c, want_s = ref.route_batch(ap, ad)
    choice = choice.cpu().numpy()
    assert (choice == want_c).all(), f"first difference at arrival {int(np.argmax(choice != want_c))}"
    assert_scores_close(score.cpu().numpy(), want_s, want_c)
    assert_state_equal(st, ref, f"after routing config {idx}")
    assert st.status() == B.PRE_OK
    st.close()


ROUTE_SHAPES = [(21, 1, 5, 10, 6), (22, 3, 9, 30, 25), (23, 7, 16, 60, 40), (24, 4, 1, 20, 10),
                (25, 6, 40, 0, 30), (26, 200, 7, 500, 300), (27, 150, 64, 2000, 200), (28, 5, 1001, 300, 100),
                (29, 333, 130, 3000, 257), (30, 6, 4100, 200, 60), (34, 3, 8190, 100, 40), (36, 9000, 6, 20000, 300),
                (37, 12000, 4, 20000, 200)]


@pytest.mark.parametrize("seed,n_inst,h,n,a", ROUTE_SHAPES)
def test_route_shapes(seed, n_inst, h, n, a, router):
    wl = W.make_random(seed, n_inst, h, n, a, max_prompt=300, max_output=2 * h + 3)
    st, ref = both(wl)
    ap, ad = wl.ticks[0]
    choice, score = st.route_batch(dev(ap), dev(ad))
    want_c, want_s = ref.route_batch(ap, ad)
    assert (choice.cpu().numpy() == want_c).all()
    assert_scores_close(score.cpu().numpy(), want_s, want_c)
    assert_state_equal(st, ref)
    st.close()


@pytest.mark.parametrize("max_prompt,n", [(2 ** 27, 6000), (2 ** 24, 18000), (2 ** 24, 20000), (2 ** 20, 40000)])
def test_route_values_around_and_above_32_bits(max_prompt, n, router):
    """Rows whose cells cross 2^32 during the batch, start above it, or stay below it."""
    wl = W.make_random(35, 40, 128, n, 400, max_prompt=max_prompt, max_output=300, capacity=10 ** 9)
    st, ref = both(wl)
    ap, ad = wl.ticks[0]
    ap = (ap.astype(np.int64) * 4000 % (2 ** 27)).astype(np.int32)   # heavy arrivals push rows over the edge
    choice, score = st.route_batch(dev(ap), dev(ad))
    want_c, want_s = ref.route_batch(ap, ad)
    assert (choice.cpu().numpy() == want_c).all()
    assert_scores_close(score.cpu().numpy(), want_s, want_c)
    assert_state_equal(st, ref)
    st.close()


def test_route_fractional_threshold_and_beta_without_score_output(router):
    wl = W.make_random(31, 50, 24, 800, 300, capacity=33337, beta=0.75)
    wl.t_mem = 0.8
    st, ref = both(wl)
    ap, ad = wl.ticks[0]
    choice, score = st.route_batch(dev(ap), dev(ad), want_score=False)
    want_c, _ = ref.route_batch(ap, ad)
    assert score is None and (choice.cpu().numpy() == want_c).all()
    assert_state_equal(st, ref)
    st.close()


def test_route_consecutive_batches_and_empty_batch(router):
    wl = W.make_random(32, 40, 32, 500, 400)
    wl.max_requests = 500 + 400
    st, ref = both(wl)
    ap, ad = wl.ticks[0]
    got, want = [], []
    for lo, hi in [(0, 1), (1, 1), (1, 130), (130, 131), (131, 400)]:
        c, _ = st.route_batch(dev(ap[lo:hi]), dev(ad[lo:hi]))
        got.append(c.cpu().numpy())
        want.append(ref.route_batch(ap[lo:hi], ad[lo:hi])[0])
    assert (np.concatenate(got) == np.concatenate(want)).all()
    assert_state_equal(st, ref)
    st.close()


def test_route_table_full_and_malformed_arrivals(router):
    wl = W.make_random(33, 6, 16, 100, 20)
    wl.max_requests = 100 + 12
    st, ref = both(wl)
    ap, ad = wl.ticks[0][0].copy(), wl.ticks[0][1].copy()
    ad[3] = 0
    ap[5] = -4
    choice, _ = st.route_batch(dev(ap), dev(ad))
    want_c, _ = ref.route_batch(ap, ad)
    assert (choice.cpu().numpy() == want_c).all()
    assert_state_equal(st, ref)
    assert st.status() == B.PRE_ECAPACITY        # the most severe of the two recorded conditions
    st.close()
    wl.max_requests = 100 + 20
    st, ref = both(wl)
    choice, _ = st.route_batch(dev(ap), dev(ad))
    assert (choice.cpu().numpy() == ref.route_batch(ap, ad)[0]).all()
    assert st.status() == B.PRE_EBADREQ
    st.close()


def test_route_large_prefix_against_literal_oracle(router):
    """Largest configuration, launch shape of the benchmark; the literal oracle on the first arrivals."""
    wl = W.make_config(3)
    st, ref = both(wl)
    ap, ad = wl.ticks[0][0][:192], wl.ticks[0][1][:192]
    choice, score = st.route_batch(dev(ap), dev(ad))
    want_c, want_s = ref.route_batch(ap, ad)
    assert (choice.cpu().numpy() == want_c).all()
    assert_scores_close(score.cpu().numpy(), want_s, want_c)
    assert_state_equal(st, ref)
    st.close()


@pytest.mark.slow
def test_route_large_full_batch(router):
    """All 65,536 decisions of the largest configuration.

    Expected values come from the oracle's identity mode, which the CPU tests admit only
    because it reproduces the literal mode bit for bit; on top of that, sampled decisions
    are re-scored one by one with the literal scan from a state rebuilt by the oracle.
    """
    wl = W.make_config(3)
    st, ref = both(wl)
    ap, ad = wl.ticks[0]
    choice, score = st.route_batch(dev(ap), dev(ad))
    choice, score = choice.cpu().numpy(), score.cpu().numpy()
    want_c, want_s = ref.route_batch(ap, ad, fast=True)
    assert (choice == want_c).all(), f"first difference at arrival {int(np.argmax(choice != want_c))}"
    assert_scores_close(score, want_s, want_c)
    assert_state_equal(st, ref)
    n0 = wl.n_requests
    for k in [1, 4097, 30000, 65535]:
        probe = oracle.State(wl.n_instances, wl.horizon, wl.capacity_tokens,
                             np.concatenate([wl.prompt, ap[:k]]), np.concatenate([wl.generated, np.zeros(k, np.int32)]),
                             np.concatenate([wl.predicted, ad[:k]]), np.concatenate([wl.instance, choice[:k]]),
                             n0 + k)
        probe.anticipate()
        probe.queued_p[:] = np.bincount(choice[:k], weights=ap[:k], minlength=wl.n_instances).astype(np.int64)
        s_all, _ = probe.score_all(int(ap[k]), int(ad[k]))
        assert int(np.argmin(s_all)) == int(choice[k]) and s_all.min() == score[k]
    st.close()


# ------------------------------------------------------------------ decode step

@pytest.mark.parametrize("seed,n_inst,h,n", [(41, 3, 6, 60), (42, 5, 16, 300), (43, 2, 1, 40), (44, 4, 80, 500),
                                             (45, 70, 1030, 2000), (46, 9000, 8, 30000)])
def test_step_shapes(seed, n_inst, h, n):
    wl = W.make_random(seed, n_inst, h, n, 0, max_output=2 * h + 9)
    st, ref = both(wl)
    for k in range(12):
        st.step()
        ref.step()
        assert_state_equal(st, ref, f"after step {k + 1}")
    # the table alone reproduces the maps
    keep = st.curves.clone()
    st.anticipate()
    assert torch.equal(keep, st.curves)
    assert st.status() == B.PRE_OK
    st.close()


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_route_then_step_configs(idx, router):
    wl = W.make_config(idx)
    st, ref = both(wl)
    ap, ad = wl.ticks[0]
    st.route_batch(dev(ap), dev(ad))
    ref.route_batch(ap, ad, fast=True)
    for _ in range(3):
        st.step()
        ref.step()
    assert_state_equal(st, ref)
    st.close()


def run_streaming(n_ticks):
    wl = W.make_config(4, n_ticks=n_ticks)
    st, ref = both(wl)
    for t, (ap, ad) in enumerate(wl.ticks):
        st.step()
        ref.step()
        c, s = st.route_batch(dev(ap), dev(ad))
        wc, ws = ref.route_batch(ap, ad, fast=True)
        c = c.cpu().numpy()
        assert (c == wc).all(), f"tick {t}: first difference at arrival {int(np.argmax(c != wc))}"
        assert_scores_close(s.cpu().numpy(), ws, wc)
    assert_state_equal(st, ref, "at the end of the stream")
    assert st.status() == B.PRE_OK
    st.close()


def test_streaming_config_first_ticks():
    run_streaming(12)


@pytest.mark.slow
def test_streaming_config_with_a_burst():
    run_streaming(101)


@pytest.mark.slow
def test_streaming_config_all_ticks():
    """The whole streaming configuration: 1,000 ticks, about 4.2 million routed arrivals."""
    run_streaming(1000)


# ------------------------------------------------------------------ scaler signals (Sec. 4.3.2)

def check_scaler(st, ref, **kw):
    over, row_max, summary = st.scaler_signals(**kw)
    w_over, w_max, w_sum = ref.scaler_signals(**kw)
    assert (over.cpu().numpy() == w_over).all()
    assert (row_max.cpu().numpy() == w_max).all()
    assert summary.cpu().numpy().tolist() == w_sum.tolist()
    return w_sum


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_scaler_signals_configs(idx):
    wl = W.make_config(idx)
    st, ref = both(wl)
    total = check_scaler(st, ref)
    assert total[1] > 0                      # the configurations are busy: the scale-down action may not fire
    check_scaler(st, ref, overload_level=0.7, overload_share=0.5, idle_level=0.9)
    st.close()


@pytest.mark.parametrize("seed,n_inst,h,n", [(81, 1, 1, 3), (82, 5, 63, 200), (83, 33, 130, 900), (84, 700, 8, 4000),
                                             (85, 9, 4100, 500)])
def test_scaler_signals_shapes(seed, n_inst, h, n):
    wl = W.make_random(seed, n_inst, h, n, 0, max_prompt=300, max_output=2 * h + 3)
    st, ref = both(wl)
    cap = int(np.percentile(ref.curves.max(axis=1), 50)) + 1
    for s in (st, ):
        s.close()
    wl.capacity_tokens = cap
    st, ref = both(wl)
    check_scaler(st, ref)
    check_scaler(st, ref, overload_level=0.5, overload_share=0.0, idle_level=0.3)
    assert B.pre_scaler_signals(st.ctx, st.curves, 0.95, 0.10, 0.30, None, st.current_d, st.current_d) == B.PRE_EINVAL
    st.close()


# ------------------------------------------------------------------ misprediction refinement (Sec. 4.3.1)

def refine_both(st, ref, actual_dev, actual_host, what=""):
    got = st.refine(actual_dev)
    want = ref.refine(actual_host)
    assert got.cpu().numpy().tolist() == want.tolist(), f"event counts differ {what}"
    return want


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_refine_configs_over_ticks(idx):
    """Ticks of step + refinement on the one-shot configurations after their batch was routed."""
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
        st.step()
        ref.step()
        events += refine_both(st, ref, actual_dev, actual, f"tick {t}")
        if t % 6 == 5:
            assert_state_equal(st, ref, f"after tick {t}")
    assert_state_equal(st, ref, "at the end")
    assert events[0] > 0 and events[1] > 0 and events[2] == 0
    # the maps still are what the build gives on the refined table
    after = st.curves.clone()
    st.anticipate()
    assert (st.curves == after).all()
    assert st.status() == B.PRE_OK
    st.close()


@pytest.mark.parametrize("seed,n_inst,h,n", [(91, 1, 1, 5), (92, 3, 7, 70), (93, 9, 40, 1000), (94, 130, 33, 5000),
                                             (95, 2, 300, 64)])
def test_refine_shapes_to_completion(seed, n_inst, h, n):
    wl = W.make_random(seed, n_inst, h, n, 0, max_prompt=50, max_output=40)
    err = np.rint((W.Stream(seed, 7).uniform(n) - 0.5) * 30).astype(np.int32)
    actual = np.maximum(1, wl.predicted + err).astype(np.int32)        # some real ends already lie behind
    actual_dev = dev(actual)
    st, ref = both(wl)
    refine_both(st, ref, actual_dev, actual, "before the first tick")
    assert_state_equal(st, ref, "before the first tick")
    for t in range(int(actual.max()) + 2):
        st.step()
        ref.step()
        refine_both(st, ref, actual_dev, actual, f"tick {t}")
    assert_state_equal(st, ref, "at the end")
    assert not ref.curves.any()
    assert (st.predicted[:n].cpu().numpy() == np.maximum(actual, wl.generated)).all()
    st.close()


def test_refine_many_events_on_one_row_and_beyond_the_window():
    """Every request on one instance, all ending at once, ramps longer than the window."""
    n, h = 3000, 16
    prompt = np.full(n, 1000, np.int32)
    predicted = (np.arange(n) % 200 + 50).astype(np.int32)
    generated = np.full(n, 10, np.int32)
    wl = W.make_random(5, 2, h, n, 0)
    wl.prompt, wl.generated, wl.predicted = prompt, generated, predicted
    wl.instance = np.zeros(n, np.int32)
    st, ref = both(wl)
    actual = np.full(n, 3, np.int32)
    counts = refine_both(st, ref, dev(actual), actual)
    assert counts.tolist() == [n, 0, 0]
    assert_state_equal(st, ref)
    assert not ref.curves.any()
    st.close()


def test_refine_malformed_rows_and_no_counts():
    wl = W.make_random(6, 4, 12, 200, 0)
    actual = np.maximum(1, wl.predicted - 3).astype(np.int32)
    actual[5] = 0                                   # malformed: real length below 1
    bad_inst = wl.instance.copy()
    bad_inst[9] = 77                                # malformed row in the table
    wl.instance = bad_inst
    st, ref = both(wl)
    assert st.status() == B.PRE_EBADREQ             # the build already reports row 9
    for _ in range(6):
        st.step()
        ref.step()
        assert st.refine(dev(actual), want_counts=False) is None
        ref.refine(actual)
    assert_state_equal(st, ref)
    assert st.status() == B.PRE_EBADREQ
    st.close()


def test_refine_streaming_ticks():
    """The streaming configuration with real lengths: step, refinement, then the tick's arrivals."""
    wl = W.make_config(4, n_ticks=16)
    table_actual, tick_actual = W.make_actual(wl, W.BASE_SEED + 4)
    st, ref = both(wl)
    actual = np.zeros(wl.max_requests, np.int32)
    actual[: len(table_actual)] = table_actual
    filled = len(table_actual)
    actual_dev = dev(actual)
    for t, (ap, ad) in enumerate(wl.ticks):
        st.step()
        ref.step()
        refine_both(st, ref, actual_dev, actual, f"tick {t}")
        c, _ = st.route_batch(dev(ap), dev(ad))
        wc, _ = ref.route_batch(ap, ad, fast=True)
        assert (c.cpu().numpy() == wc).all(), f"tick {t}"
        actual[filled: filled + len(ap)] = tick_actual[t]
        actual_dev[filled: filled + len(ap)] = dev(tick_actual[t])
        filled += len(ap)
    assert_state_equal(st, ref, "at the end of the stream")
    st.close()


# ------------------------------------------------------------------ router with admission queue (Sec. 4.3.3)

def both_with_queue(wl, capacity):
    st, ref = both(wl)
    st.make_queue(capacity)
    ref.make_queue(capacity)
    return st, ref


def admit_both(st, ref, ap, ad, level, share, what=""):
    """One call on both sides; compares results, the queue and the whole state."""
    waiting = int(ref.queue_state[1])
    qc, c, s = st.route_admit(dev(ap), dev(ad), overload_level=level, overload_share=share)
    wqc, wc, ws = ref.route_admit(ap, ad, overload_level=level, overload_share=share, fast=True)
    c = c.cpu().numpy()
    assert (c == wc).all(), f"{what}: first difference at arrival {int(np.argmax(c != wc))}: {c[c != wc][:4]} vs {wc[c != wc][:4]}"
    assert (qc[:waiting].cpu().numpy() == wqc).all(), f"{what}: results of the waiting requests differ"
    assert_scores_close(s.cpu().numpy(), ws, wc)
    assert (s.cpu().numpy()[wc < 0] == 0).all()
    assert st.queue_state.cpu().numpy().tolist() == ref.queue_state.tolist(), f"{what}: queue head/length differ"
    head, n = (int(v) for v in ref.queue_state)
    if n:
        idx = (head + np.arange(n)) % ref.queue_capacity
        assert (st.queue_prompt.cpu().numpy()[idx] == ref.queue_prompt[idx]).all(), f"{what}: queue contents differ"
        assert (st.queue_predicted.cpu().numpy()[idx] == ref.queue_predicted[idx]).all(), f"{what}: queue contents differ"
    assert_state_equal(st, ref, what)
    return wc


@pytest.mark.parametrize("idx,level,first_blocked", [(0, 0.6, 25), (1, 0.6, 335), (2, 0.3, 5979), (1, 0.95, None),
                                                     (0, 0.3, 0)])
def test_admit_configs(idx, level, first_blocked, router):
    wl = W.make_config(idx)
    st, ref = both_with_queue(wl, 100)
    ap, ad = wl.ticks[0]
    c = admit_both(st, ref, ap, ad, level, 0.10, f"config {idx}")
    if first_blocked is None:
        assert (c >= 0).all()
    else:
        assert (c[:first_blocked] >= 0).all() and (c[first_blocked:] < 0).all()
    assert st.status() == B.PRE_OK
    st.close()


def test_admit_never_blocking_equals_route_batch(router):
    wl = W.make_config(1)
    st, ref = both_with_queue(wl, 10)
    plain = DeviceState.from_workload(wl)
    plain.anticipate()
    ap, ad = wl.ticks[0]
    _, c, s = st.route_admit(dev(ap), dev(ad), overload_level=1e9)
    pc, ps = plain.route_batch(dev(ap), dev(ad))
    assert (c == pc).all() and (s == ps).all() and (st.curves == plain.curves).all()
    st.close()
    plain.close()


@pytest.mark.parametrize("seed,n_inst,h,n,a,qcap,level", [(11, 3, 8, 30, 40, 5, 0.7), (12, 2, 5, 10, 30, 0, 0.7),
                                                          (13, 5, 16, 80, 60, 100, 0.5), (14, 1, 4, 6, 12, 3, 0.9),
                                                          (15, 4, 12, 50, 64, 7, 0.7), (16, 300, 64, 4000, 900, 64, 0.8),
                                                          (17, 149, 128, 3000, 700, 1000, 0.75)])
def test_admit_shapes_over_several_calls(seed, n_inst, h, n, a, qcap, level, router):
    """Calls alternate with decode steps: requests wait, are routed later, the ring's head moves on."""
    wl = W.make_random(seed, n_inst, h, n, a, max_prompt=30, max_output=20)
    st, ref = both_with_queue(wl, qcap)
    ap, ad = wl.ticks[0]
    seen = set()
    for call in range(4):
        lo, hi = call * a // 4, (call + 1) * a // 4
        c = admit_both(st, ref, ap[lo:hi], ad[lo:hi], level, 0.25, f"call {call}")
        seen |= set(np.sign(c).tolist()) | set(c[c < 0].tolist())
        for _ in range(3):
            st.step()
            ref.step()
    assert_state_equal(st, ref, "at the end")
    if seed < 16:
        assert 1 in seen or 0 in seen
        assert -2 in seen or -3 in seen
    st.close()


def test_admit_long_tail_after_the_block_and_malformed_arrivals(router):
    """Thousands of arrivals behind the blocked one: they join the queue in order until it is full."""
    wl = W.make_config(2)
    st, ref = both_with_queue(wl, 1500)
    ap, ad = (x.copy() for x in wl.ticks[0])
    ap[6000] = -5                       # malformed, beyond the point where the batch blocks
    ad[7000] = 0
    ap[17] = -1                         # malformed, before it
    c = admit_both(st, ref, ap, ad, 0.3, 0.10, "first call")
    assert c[17] == -1 and c[6000] == -1 and c[7000] == -1
    assert (c == -2).sum() == 1500 and (c == -3).sum() > 0
    assert st.status() == B.PRE_EBADREQ
    # nothing drains: a second call changes nothing but the results
    c = admit_both(st, ref, ap[:10], ad[:10], 0.3, 0.10, "second call")
    assert (c == -3).all()
    # 200 steps later the queue drains (in order) before the new arrivals
    for _ in range(200):
        st.step()
        ref.step()
    admit_both(st, ref, ap[:64], ad[:64], 0.3, 0.10, "third call")
    st.close()


def test_admit_table_full_and_empty_call(router):
    wl = W.make_random(31, 4, 16, 20, 12)
    wl.max_requests = 25
    st, ref = both_with_queue(wl, 8)
    ap, ad = wl.ticks[0]
    c = admit_both(st, ref, ap, ad, 1e9, 0.1, "table fills")
    assert (c[:5] >= 0).all() and (c[5:] == -1).all()
    assert st.status() == B.PRE_ECAPACITY
    admit_both(st, ref, ap[:0], ad[:0], 1e9, 0.1, "empty call")
    st.close()

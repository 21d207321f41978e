"""The single-launch anticipator build: every way it can lay out and accumulate a table.

The lists of a build are placed where the previous build's list lengths suggest (with spare room), and
exactly, from the totals, when a piece does not fit; tiles are accumulated in compact 32-bit cells,
in 64-bit cells when those overflow, and in the wide mode when 32-bit sums do not suffice; tables whose
largest B needs more than 19 bits take 8-byte records; tables beyond the launch's capacity take the
two-kernel build.  Every case is compared with the oracle (the definition of Sec. 4.3.1 written out),
bit for bit, on several calls in a row on one context.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2504_03702_b200 import binding as B  # noqa: E402
from paper_2504_03702_b200 import workloads as W  # noqa: E402
from paper_2504_03702_b200.state import DeviceState  # noqa: E402


def expect(prompt, generated, predicted, instance, n_inst, h):
    ref = oracle.State(n_inst, h, 1000, prompt, generated, predicted, instance, len(prompt))
    ref.anticipate()
    return ref.curves, ref.current_d


def check(st, table, n_inst, h, what):
    st.load_requests(*table)
    st.curves.fill_(-3)
    st.current_d.fill_(-3)
    st.anticipate()
    assert st.status() == B.PRE_OK, what
    want_c, want_d = expect(*table, n_inst, h)
    got = st.curves.cpu().numpy()
    assert (got == want_c).all(), f"{what}: {int((got != want_c).sum())} cells differ"
    assert (st.current_d.cpu().numpy() == want_d).all(), what


def table_of(wl, n=None):
    n = wl.n_requests if n is None else n
    return wl.prompt[:n], wl.generated[:n], wl.predicted[:n], wl.instance[:n]


def test_same_table_then_changed_tables_on_one_context():
    n_inst, h = 96, 1024
    big = W.make_random(301, n_inst, h, 60000, 0, max_prompt=4000, max_output=3000)
    other = W.make_random(302, n_inst, h, 60000, 0, max_prompt=4000, max_output=3000)
    layout = DeviceState(n_inst, h, 1000, 60000)
    code, info = B.pre_query_layout(layout.ctx)
    assert code == B.PRE_OK and info[2] > 0 and info[3] >= 60000, "this shape is meant to take the single-launch build"
    layout.close()
    st = DeviceState(n_inst, h, 1000, 60000)
    check(st, table_of(big), n_inst, h, "first build (lists laid out exactly)")
    check(st, table_of(big), n_inst, h, "same table (lists where the first build's lengths put them)")
    check(st, table_of(big), n_inst, h, "same table again")
    check(st, table_of(other), n_inst, h, "another table of the same size")
    check(st, table_of(big, 20000), n_inst, h, "a third of the table")
    check(st, table_of(big, 21000), n_inst, h, "a little more (inside the spare room)")
    check(st, table_of(big), n_inst, h, "three times as much (outside the spare room)")
    skew = big.instance.copy()
    skew[: 40000] = 5                                        # most requests on one instance
    check(st, (big.prompt, big.generated, big.predicted, skew), n_inst, h, "skewed assignment")
    check(st, (big.prompt, big.generated, big.predicted, skew), n_inst, h, "skewed assignment again")
    check(st, table_of(big, 0), n_inst, h, "empty table")
    check(st, table_of(big), n_inst, h, "after the empty table")
    st.close()


def test_cells_that_overflow_the_compact_words():
    # thousands of requests end at the same step of the same row: more than a compact cell counts,
    # and sums of B beyond its 20 bits
    n_inst, h, n = 8, 512, 30000
    rs = np.random.RandomState(5)
    prompt = rs.randint(100, 3000, n).astype(np.int32)
    generated = np.zeros(n, np.int32)
    predicted = rs.randint(1, 600, n).astype(np.int32)
    instance = rs.randint(0, n_inst, n).astype(np.int32)
    predicted[:9000] = 77
    instance[:9000] = 3
    prompt[9000:9400] = 200000            # a few long prompts in one cell: few records, large sum
    predicted[9000:9400] = 12
    instance[9000:9400] = 6
    st = DeviceState(n_inst, h, 1000, n)
    for k in range(3):
        check(st, (prompt, generated, predicted, instance), n_inst, h, f"call {k}")
    st.close()


def test_eight_byte_records_and_wide_sums():
    n_inst, h, n = 40, 512, 20000
    rs = np.random.RandomState(6)
    prompt = rs.randint(1, 1 << 22, n).astype(np.int32)       # B needs more than 19 bits
    generated = rs.randint(0, 50, n).astype(np.int32)
    predicted = (generated + rs.randint(1, 700, n)).astype(np.int32)
    instance = rs.randint(0, n_inst, n).astype(np.int32)
    st = DeviceState(n_inst, h, 1000, n)
    for k in range(2):
        check(st, (prompt, generated, predicted, instance), n_inst, h, f"8-byte records, call {k}")
    small = np.minimum(prompt, 3000)
    check(st, (small, generated, predicted, instance), n_inst, h, "4-byte records after 8-byte records")
    check(st, (small, generated, predicted, instance), n_inst, h, "4-byte records again")
    huge = prompt.copy()
    huge[:] = (1 << 27) - 100                                  # sums beyond 32 bits: the wide mode
    check(st, (huge, generated, predicted, instance), n_inst, h, "wide sums")
    check(st, (small, generated, predicted, instance), n_inst, h, "narrow again")
    st.close()


def test_lists_longer_than_one_bulk_copy():
    n_inst, h, n = 4, 2048, 40000                              # one tile receives every request
    wl = W.make_random(303, n_inst, h, n, 0, max_prompt=3000, max_output=4000)
    st = DeviceState(n_inst, h, 1000, n)
    for k in range(2):
        check(st, table_of(wl), n_inst, h, f"call {k}")
    st.close()


@pytest.mark.slow
def test_table_beyond_the_single_launch_build():
    n_inst, h = 256, 64
    st = DeviceState(n_inst, h, 1000, 2_400_000)
    code, info = B.pre_query_layout(st.ctx)
    n = info[3] + 4096                                         # more rows than the single launch takes
    assert n <= 2_400_000
    wl = W.make_random(304, n_inst, h, n, 0, max_prompt=500, max_output=90)
    check(st, table_of(wl), n_inst, h, "two-kernel build")
    check(st, table_of(wl, info[3]), n_inst, h, "single launch at its largest table")
    check(st, table_of(wl), n_inst, h, "two-kernel build again")
    st.close()

"""pre_anticipate_static: the build for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits: inside a serving engine whose
pool allocator owns the whole GPU, under the allocator's lock, or in a control loop that must
not risk the device-wide synchronisation an allocation can bring.  For them the library
carries its scratch inside its own image and exposes one entry point that needs no context.
This file checks, through the C-ABI, that it computes exactly what pre_anticipate computes
(int64 maps and backlogs, bit for bit) and what the CPU oracle computes, on calls in a row that
share the built-in scratch, and that it refuses problems larger than that scratch.  (The allocation
check sees torch's allocator only; that the entry point itself requests no memory is a property of
its source, which calls no allocating routine.)

It is collected last on purpose (see conftest.py): if it fails, every other test has run.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
from paper_2504_03702_b200 import binding as B  # noqa: E402
from paper_2504_03702_b200 import workloads as W  # noqa: E402
from paper_2504_03702_b200.state import DeviceState  # noqa: E402


def with_context(wl):
    st = DeviceState.from_workload(wl)
    st.anticipate()
    assert st.status() == B.PRE_OK
    out = st.curves.clone(), st.current_d.clone()
    return st, out


def without_allocation(st, wl, curves, current_d, flags):
    """The caller still owns inputs and outputs; they are allocated before the call under test."""
    flags.zero_()
    code = B.pre_anticipate_static(wl.n_instances, wl.horizon, st.prompt, st.generated, st.predicted,
                                   st.instance, wl.n_requests, curves, current_d, flags)
    assert code == B.PRE_OK, B.pre_strerror(code)
    torch.cuda.synchronize()


def test_two_calls_in_a_row_match_the_context_path():
    first = W.make_config(1)                                   # 64 instances, H = 256, 16,384 requests
    second = W.make_random(91, 300, 96, 50000, 0, max_prompt=3000, max_output=400)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    for wl in (first, second, first):                          # the third call sees the second's leftovers
        st, (want_curves, want_d) = with_context(wl)
        curves = torch.full_like(want_curves, -7)
        current_d = torch.full_like(want_d, -7)
        before = torch.cuda.memory_allocated()
        without_allocation(st, wl, curves, current_d, flags)
        assert torch.cuda.memory_allocated() == before
        assert torch.equal(curves, want_curves)
        assert torch.equal(current_d, want_d)
        assert int(flags.item()) == 0
        # and both against the definition written out on the CPU, not only against each other
        ref = oracle.State.from_workload(wl)
        ref.anticipate()
        assert (curves.cpu().numpy() == ref.curves).all()
        assert (current_d.cpu().numpy() == ref.current_d).all()
        st.close()


def test_malformed_requests_are_flagged_and_empty_tables_work():
    wl = W.make_random(92, 20, 64, 2000, 0)
    wl.instance[5] = 99
    wl.predicted[6] = 0
    st = DeviceState.from_workload(wl)
    st.anticipate()
    assert st.status() == B.PRE_EBADREQ
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    curves = torch.empty_like(st.curves)
    current_d = torch.empty_like(st.current_d)
    without_allocation(st, wl, curves, current_d, flags)
    assert torch.equal(curves, st.curves) and torch.equal(current_d, st.current_d)
    assert int(flags.item()) != 0
    code = B.pre_anticipate_static(wl.n_instances, wl.horizon, None, None, None, None, 0, curves, current_d, None)
    assert code == B.PRE_OK
    torch.cuda.synchronize()
    assert int(curves.abs().sum()) == 0 and int(current_d.abs().sum()) == 0
    st.close()


def test_sizes_beyond_the_built_in_scratch_are_refused():
    curves = torch.zeros(16, dtype=torch.int64, device="cuda")
    d = torch.zeros(4, dtype=torch.int64, device="cuda")
    req = torch.zeros(8, dtype=torch.int32, device="cuda")
    too_many = B.pre_anticipate_static(4, 4, req, req, req, req, 262144 + 1, curves, d, None)
    assert too_many == B.PRE_ESIZE and "built-in scratch" in B.pre_strerror(too_many)
    # 16,384 x 2,048 cells need 8,192 tiles: more than the scratch indexes (nothing is launched)
    assert B.pre_anticipate_static(16384, 2048, req, req, req, req, 8, curves, d, None) == B.PRE_ESIZE
    assert B.pre_anticipate_static(4, 0, req, req, req, req, 8, curves, d, None) == B.PRE_EINVAL
    assert B.pre_anticipate_static(4, 4, req, req, req, req, 8, None, d, None) == B.PRE_EINVAL
    torch.cuda.synchronize()

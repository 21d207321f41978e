"""Helpers for the GPU parity tests: run a workload through the C-ABI, mirror it in the oracle."""
import numpy as np
import torch

import oracle
from paper_2504_03702_b200 import binding as B
from paper_2504_03702_b200.state import DeviceState


def dev(a, dtype=np.int32):
    return torch.as_tensor(np.ascontiguousarray(a, dtype=dtype)).cuda()


def table(st: DeviceState):
    n = st.sync_count()
    return [t[:n].cpu().numpy() for t in (st.prompt, st.generated, st.predicted, st.instance)]


def assert_state_equal(st: DeviceState, ref: oracle.State, what=""):
    assert (st.curves.cpu().numpy() == ref.curves).all(), f"curves differ {what}"
    assert (st.current_d.cpu().numpy() == ref.current_d).all(), f"current_d differs {what}"
    assert (st.queued_p.cpu().numpy() == ref.queued_p).all(), f"queued_p differs {what}"
    n = st.sync_count()
    assert n == int(ref.n[0]), f"request count differs {what}"
    for got, want, name in zip(table(st), (ref.prompt, ref.generated, ref.predicted, ref.instance),
                               ("prompt", "generated", "predicted", "instance")):
        assert (got == want[:n]).all(), f"table column {name} differs {what}"


def assert_scores_close(got, want, choice):
    got, want = np.asarray(got), np.asarray(want)
    ok = choice >= 0
    rel = np.abs(got[ok] - want[ok]) / np.maximum(np.abs(want[ok]), 1.0)
    assert rel.size == 0 or rel.max() <= 1e-12, f"score off by {rel.max()} relative"

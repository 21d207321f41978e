"""The N > 1 timing protocol (barrier, max over ranks, aggregate) on two gloo ranks on CPU."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    from paper_2504_03702_b200 import dist as D
    g = D.init(world, rank, backend="gloo")
    D.barrier(g)
    local_ms = 10.0 + 5.0 * rank            # rank 1 is the slow replica
    slowest = D.max_over_ranks(local_ms, g)
    agg = D.aggregate_throughput(1000.0, local_ms, world, g)
    out.put((rank, slowest, agg))
    D.finish(g)


def test_two_rank_timing_protocol():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, agg in got:
        assert slowest == 15.0
        assert abs(agg - 2 * 1000.0 / 15e-3) < 1e-6


def test_single_process_needs_no_group():
    from paper_2504_03702_b200 import dist as D
    assert D.init(1, 0) is None
    assert D.max_over_ranks(3.5, None) == 3.5
    D.barrier(None)
    D.finish(None)

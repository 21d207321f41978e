"""Process-group plumbing for runs on several GPUs of one node.

The path does not shard without an exchange per arrival (every arrival must see every
instance's score), and one GPU holds the largest configuration many times over, so more
GPUs run independent replicas: one service per GPU, no data-path collective.  The only
communication is the timing protocol: a barrier on both sides of the timed region and the
maximum of the per-rank times.
"""
from __future__ import annotations

import os


def init(world: int, rank: int, backend: str = "nccl", device=None):
    """Returns a handle (None for a single process)."""
    if world <= 1:
        return None
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29531")
    kwargs = {}
    if backend == "nccl" and device is not None:
        kwargs["device_id"] = device
    dist.init_process_group(backend=backend, rank=rank, world_size=world, **kwargs)
    return dist


def barrier(group):
    if group is not None:
        group.barrier()


def max_over_ranks(value: float, group, device=None) -> float:
    """Largest `value` over all ranks (the job is as slow as its slowest replica)."""
    if group is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    group.all_reduce(t, op=group.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, ms_local: float, world: int, group, device=None) -> float:
    """Whole-job units per second: every rank processed `units_per_rank` in at most max-over-ranks ms."""
    ms = max_over_ranks(ms_local, group, device)
    return world * units_per_rank / (ms * 1e-3)


def finish(group):
    if group is not None:
        group.barrier()
        group.destroy_process_group()

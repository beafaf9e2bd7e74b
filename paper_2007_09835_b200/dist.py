"""Process-group plumbing for batch-sharded replicas (one process per GPU).

The convolution path shards over the batch dimension with no exchange step: every rank
holds a replica of the packed weights and runs its own clips.  The only collectives are
the barrier and the max-reduce of timings used by the benchmark; they work on the `nccl`
backend (GPU) and on `gloo` (CPU tests).
"""
from __future__ import annotations

import datetime
import os


def init(world_size: int, rank: int, backend: str = "nccl"):
    """Initialise the default process group from MASTER_ADDR / MASTER_PORT; returns the group."""
    import torch.distributed as td
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    if not td.is_initialized():
        td.init_process_group(backend, rank=rank, world_size=world_size,
                              timeout=datetime.timedelta(seconds=300))
    return td.group.WORLD


def barrier(group):
    if group is not None:
        import torch.distributed as td
        td.barrier(group=group)


def max_over_ranks(value: float, group, device=None) -> float:
    """Largest `value` over all ranks of the group (the slowest rank decides a timing)."""
    if group is None:
        return float(value)
    import torch
    import torch.distributed as td
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    td.all_reduce(t, op=td.ReduceOp.MAX, group=group)
    return float(t.item())


def sum_over_ranks(value: float, group, device=None) -> float:
    if group is None:
        return float(value)
    import torch
    import torch.distributed as td
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    td.all_reduce(t, op=td.ReduceOp.SUM, group=group)
    return float(t.item())


def shard_clips(n_clips: int, world_size: int, rank: int) -> range:
    """Contiguous block of clip indices owned by `rank` (sizes differ by at most one)."""
    base, extra = divmod(n_clips, world_size)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def aggregate_throughput(local_units: float, local_ms: float, group, device=None) -> float:
    """Whole-job throughput: units processed by all ranks / slowest rank's time (units per second)."""
    total = sum_over_ranks(local_units, group, device)
    ms = max_over_ranks(local_ms, group, device)
    return total / (ms * 1e-3)


def shutdown(group):
    if group is not None:
        import torch.distributed as td
        if td.is_initialized():
            td.destroy_process_group()

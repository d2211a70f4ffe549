"""Rank bookkeeping for `bench.py --gpus N`.

The hot path does not shard: every step is sample-local and the benchmark fixes one GPU per batch, so
N GPUs run N independent replicas with no data-path collective.  The only communication is timing:
a barrier on both sides of the timed region and the maximum of the per-rank elapsed times; the
reported value is the units all ranks processed divided by that maximum.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def world_info():
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar (elapsed milliseconds) over all ranks."""
    rank, world = world_info()
    if world == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, local_ms: float, device="cpu") -> float:
    """Whole-job units per second: every rank processed `units_per_rank` in at most max(local_ms)."""
    _, world = world_info()
    ms = max_over_ranks(local_ms, device)
    return world * units_per_rank / (ms * 1e-3)

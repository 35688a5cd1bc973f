"""Process-group plumbing for running independent replicas, one process per GPU.

The decoding stream of one query is a strictly sequential chain of forwards (the paper's setting is a single
query), so ranks exchange nothing on the data path.  The group exists for the start barrier and for taking
the slowest rank's time."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def init(world: int, rank: int, backend: str):
    if world <= 1:
        return None
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29533")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend, world_size=world, rank=rank)
    return dist.group.WORLD


def _dev(group):
    return "cuda" if group is not None and dist.get_backend(group) == "nccl" else "cpu"


def barrier(group):
    if group is not None:
        t = torch.zeros(1, device=_dev(group))
        dist.all_reduce(t, group=group)
        if t.is_cuda:
            torch.cuda.synchronize()


def max_over_ranks(x: float, group) -> float:
    if group is None:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=_dev(group))
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def sum_over_ranks(x: float, group) -> float:
    if group is None:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=_dev(group))
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return float(t.item())


def aggregate_throughput(units_this_rank: float, ms_this_rank: float, group) -> float:
    """Whole-job rate: units of all ranks over the slowest rank's time (units per second)."""
    return sum_over_ranks(units_this_rank, group) / (max_over_ranks(ms_this_rank, group) * 1e-3)


def finish(group):
    if group is not None and dist.is_initialized():
        dist.destroy_process_group()

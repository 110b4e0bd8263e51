"""Multi-rank plumbing for the benchmark: one process per GPU over ``torch.distributed``.

The hot path shards by batch with no data-path exchange: every (sequence, KV-head group) of the
attention forward, backward and decode is independent, and the donor-group dK/dV sum runs over
layers and heads inside one sequence.  Under batch sharding the only real exchange of a training
step is the sum of the weight gradients over ranks, done here with one all-reduce per step on a
flat fp32 bucket (NCCL on GPUs, gloo in the CPU tests).  Decode needs no collective.
"""
from __future__ import annotations

import os
from typing import List, Optional, Sequence

import torch
import torch.distributed as dist


def env_world() -> tuple:
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: Optional[str] = None) -> tuple:
    """Initialise the default process group from the torchrun environment (no-op for one rank).
    Returns (rank, local_rank, world_size)."""
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Every rank gets the maximum of `value` over ranks (timings are reported as the slowest rank)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def shard_range(n_units: int, rank: int, world: int) -> range:
    """Contiguous, balanced shard of n_units independent units (sequences) for this rank."""
    base, rem = divmod(n_units, world)
    start = rank * base + min(rank, rem)
    return range(start, start + base + (1 if rank < rem else 0))


class GradBucket:
    """Flat fp32 bucket holding every weight gradient of the block, so that the cross-rank sum of a
    training step is ONE all-reduce.  `views[i]` aliases the bucket and is what the kernels write."""

    def __init__(self, shapes: Sequence[Optional[tuple]], device):
        sizes = [0 if s is None else int(torch.Size(s).numel()) for s in shapes]
        self.flat = torch.empty(sum(sizes), dtype=torch.float32, device=device)
        self.views: List[Optional[torch.Tensor]] = []
        off = 0
        for s, n in zip(shapes, sizes):
            if s is None:
                self.views.append(None)
                continue
            off_al = off
            self.views.append(self.flat[off_al:off_al + n].view(s))
            off += n

    def all_reduce(self, async_op: bool = False):
        if not dist.is_initialized():
            return None
        return dist.all_reduce(self.flat, op=dist.ReduceOp.SUM, async_op=async_op)

"""Multi-rank plumbing for the benchmark: one process per GPU over ``torch.distributed``.

The hot path shards by batch with no data-path exchange: every (sequence, KV-head group) of the
attention forward, backward and decode is independent, and the donor-group dK/dV sum runs over
layers and heads inside one sequence.  Under batch sharding the only real exchange of a training
step is the sum of the weight gradients over ranks, done here on a flat fp32 bucket, either in one
all-reduce or layer by layer so that it overlaps the remaining gradient GEMMs (NCCL on GPUs, gloo in
the CPU tests).  Decode needs no collective.
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


def is_multi() -> bool:
    return dist.is_initialized() and dist.get_world_size() > 1


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
    """Flat fp32 bucket holding every weight gradient of the block; `views[i]` aliases the bucket and is what the
    kernels write.  With `layer_of` (the layer each entry belongs to) the entries of one layer are laid out
    next to each other, so that the cross-rank sum can be issued layer by layer -- each layer's slice as soon as
    its gradients are enqueued, on a side stream, leaving only the last layer's reduction exposed -- as well as
    in one piece."""

    def __init__(self, shapes: Sequence[Optional[tuple]], device, layer_of: Optional[Sequence[int]] = None):
        sizes = [0 if s is None else int(torch.Size(s).numel()) for s in shapes]
        self.flat = torch.empty(sum(sizes), dtype=torch.float32, device=device)
        self.views: List[Optional[torch.Tensor]] = [None] * len(shapes)
        order = list(range(len(shapes)))
        if layer_of is not None:
            order.sort(key=lambda i: (layer_of[i], i))
        self.layer_slices = {}
        off = 0
        for i in order:
            s, n = shapes[i], sizes[i]
            if s is None:
                continue
            self.views[i] = self.flat[off:off + n].view(s)
            if layer_of is not None:
                a, _b = self.layer_slices.get(layer_of[i], (off, off))
                self.layer_slices[layer_of[i]] = (a, off + n)
            off += n

    def all_reduce(self, async_op: bool = False):
        if not dist.is_initialized():
            return None
        return dist.all_reduce(self.flat, op=dist.ReduceOp.SUM, async_op=async_op)

    def all_reduce_layer(self, layer: int, async_op: bool = False):
        """Sum of one layer's slice over ranks (the slices of all layers partition the bucket)."""
        a, b = self.layer_slices[layer]
        if not dist.is_initialized() or a == b:
            return None
        return dist.all_reduce(self.flat[a:b], op=dist.ReduceOp.SUM, async_op=async_op)

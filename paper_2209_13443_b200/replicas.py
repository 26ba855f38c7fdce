"""Host-side plumbing of a multi-GPU run: independent replicas, one process per GPU.

Samples are independent from input to exit (convolution, pooling, FC, softmax and the threshold are
per sample; compaction and refill only permute), so the path shards by request with no collective
on the data path.  ``torch.distributed`` is used for the start/stop barrier and for the max-over-ranks
time only.  Works on any backend (``nccl`` on GPUs, ``gloo`` in the CPU tests).
"""
from __future__ import annotations


def rank_requests(rank: int, world: int, per_rank: int):
    """Request ids served by ``rank``: a contiguous block, disjoint across ranks, covering [0, world*per_rank)."""
    if not (0 <= rank < world) or per_rank < 0:
        raise ValueError("bad rank/world/per_rank")
    return rank * per_rank, per_rank


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The slowest rank's time (what a whole-job throughput must be computed from)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch

    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world: int, units_per_rank_per_step: int, steps: int, max_ms: float) -> float:
    """Whole-job units per second: everything all ranks processed over the slowest rank's time."""
    return world * units_per_rank_per_step * steps / (max_ms * 1e-3)

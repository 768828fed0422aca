"""Host-side plumbing of the multi-GPU bench: one process per GPU, each an independent
replica on its own minibatches (no data-path collective; the paper's exchange between
replicas is carried out inside one GPU's memory by alexnet_replica_average).  Only the
timing crosses ranks: the step time of the job is the maximum over ranks.

These helpers work with any torch.distributed backend (NCCL on GPUs, gloo on CPU)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_stream(rank: int) -> int:
    """Index of the synthetic data stream a rank draws its minibatches from (synth.images(seed, stream, step, B)):
    every rank trains on different data, as the paper's replicas do."""
    return int(rank)


def barrier(world: int) -> None:
    if world > 1:
        dist.barrier()


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """Maximum of a per-rank scalar (the timed milliseconds) over all ranks."""
    if world <= 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, world: int, ms: float) -> float:
    """Whole-job units per second when every rank processed units_per_rank units in ms milliseconds (the maximum)."""
    return units_per_rank * world / (ms * 1e-3)

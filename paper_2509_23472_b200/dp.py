"""Data-parallel bookkeeping of the benchmark: the hot path shards by batch and needs no collective.

In data-parallel fine-tuning every rank holds its own micro-batch of activations and compresses it on its own
GPU; nothing of Algorithm 1 crosses ranks.  What the ranks share is only how a run is laid out and reported:
which batch and which sampled rows a rank gets, and how per-rank times become one whole-job figure.  That logic
lives here, apart from any CUDA call, so that it runs (and is tested) on CPU process groups as well.
"""
from __future__ import annotations

import dataclasses
from typing import Sequence

import torch

from . import synth

SEED_STRIDE = 7919   # distance between the input seeds of consecutive ranks


def rank_workload(w: synth.Workload, rank: int) -> synth.Workload:
    """The batch of `rank`: the same recipe and shape, drawn from a seed of its own (rank 0 keeps the workload's)."""
    return dataclasses.replace(w, seed=w.seed + SEED_STRIDE * rank)


def rank_call_id(rank: int) -> int:
    """Counter word of the row sampler: replicas must not sample the same rows, so it carries the rank."""
    return rank


def max_over_ranks(values: Sequence[float], dist=None, device="cpu") -> list:
    """Element-wise maximum of per-rank timings over the process group (identity without one)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_gbs(world: int, x_bytes_per_rank: int, ms_per_step: float) -> float:
    """GB/s of X over all ranks: every rank processes its own x_bytes_per_rank in the (slowest rank's) step time."""
    return world * x_bytes_per_rank / (ms_per_step * 1e-3) / 1e9

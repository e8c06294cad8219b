"""Helpers for running independent replicas of the decode path, one process per
GPU.  The path shards by sequence with no exchange step, so the only
communication is bookkeeping: a barrier around the timed region and the maximum
of the ranks' times.  Works with any ``torch.distributed`` backend (nccl on
GPUs, gloo on CPU)."""
from __future__ import annotations

from typing import List, Sequence

import numpy as np


def shard_sequences(n_seqs: int, world: int, rank: int) -> range:
    """Contiguous share of ``n_seqs`` sequences for ``rank`` (sizes differ by at most one)."""
    lo = n_seqs * rank // world
    hi = n_seqs * (rank + 1) // world
    return range(lo, hi)


def barrier(dist=None):
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def max_over_ranks(x: float, dist=None, device: str = "cpu") -> float:
    """Largest value any rank passed; every rank gets it."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(x)
    import torch
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(seqs_per_rank: int, steps: int, max_ms: float, world: int) -> float:
    """Whole-job throughput of ``world`` replicas that each advanced ``seqs_per_rank``
    sequences by ``steps`` decode steps, the slowest taking ``max_ms``."""
    return world * seqs_per_rank * steps / (max_ms * 1e-3)

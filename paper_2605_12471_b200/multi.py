"""Multi-GPU plumbing of the benchmark: the fold step shards by independent sequences.

One process per GPU; rank r folds sequence r into its own cache.  There is no exchange on the
data path (a cache never leaves its GPU), so the only collectives are a barrier around the timed
region and the max-over-ranks of the elapsed time.  Works on any torch.distributed backend (NCCL
on GPUs, gloo on CPU for tests).
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_rank() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def sequence_of_rank(rank: int, sequences_per_rank: int = 1):
    """Sequence ids owned by a rank (contiguous blocks)."""
    return list(range(rank * sequences_per_rank, (rank + 1) * sequences_per_rank))


def max_over_ranks(value: float, device: str | torch.device = "cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank_step: int, steps: int, world: int, elapsed_ms_max: float) -> float:
    """Aggregate throughput: tokens all ranks folded / the slowest rank's time."""
    return world * steps * tokens_per_rank_step / (elapsed_ms_max * 1e-3)

"""Multi-GPU plumbing of the benchmark: the fold step shards by independent sequences, or, for
one sequence, by KV head.

One process per GPU.  By sequence: rank r folds sequence r into its own cache.  By KV head: rank
r keeps the cache planes of its block of KV heads and is given the matching query heads; since a
query head reads one KV head only, every rank's output is a disjoint slice of the heads.  Either
way there is no exchange on the data path (a cache never leaves its GPU), so the only collectives
are a barrier around the timed region and the max-over-ranks of the elapsed time.  Works on any
torch.distributed backend (NCCL on GPUs, gloo on CPU for tests).
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


def kv_head_shard(rank: int, world: int, n_q_heads: int, n_kv_heads: int) -> Tuple[range, range]:
    """(query heads, KV heads) owned by a rank when one sequence is split by KV head.

    KV heads are dealt in contiguous blocks of n_kv_heads / world; the query heads that read them
    (head h reads KV head h // (n_q_heads // n_kv_heads)) form the matching contiguous block."""
    if world < 1 or not 0 <= rank < world or n_kv_heads % world:
        raise ValueError(f"{n_kv_heads} KV heads do not split over {world} ranks")
    g = n_q_heads // n_kv_heads
    per = n_kv_heads // world
    kv = range(rank * per, (rank + 1) * per)
    return range(kv.start * g, kv.stop * g), kv


def shard_heads(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, rank: int, world: int):
    """A rank's slice of one chunk's q [n,H,d], k, v [n,Hkv,d] (contiguous copies)."""
    qh, kvh = kv_head_shard(rank, world, q.shape[-2], k.shape[-2])
    return (q[..., qh.start:qh.stop, :].contiguous(), k[..., kvh.start:kvh.stop, :].contiguous(),
            v[..., kvh.start:kvh.stop, :].contiguous())


def max_over_ranks(value: float, device: str | torch.device = "cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank_step: int, steps: int, world: int, elapsed_ms_max: float) -> float:
    """Aggregate throughput: tokens all ranks folded / the slowest rank's time."""
    return world * steps * tokens_per_rank_step / (elapsed_ms_max * 1e-3)

"""Multi-GPU plumbing of the benchmark: the fold step shards by independent sequences, or, for
one sequence, by KV head.

One process per GPU.  By sequence: rank r folds sequence r into its own cache.  By KV head: rank
r keeps the cache planes of its block of KV heads and is given the matching query heads; since a
query head reads one KV head only, every rank's output is a disjoint slice of the heads.  Either
way there is no exchange on the data path (a cache never leaves its GPU), so the only collectives
are a barrier around the timed region and the max-over-ranks of the elapsed time.

By row range (one sequence longer than one GPU's memory): chunk t is appended on rank t % world
(chunk_owner), so every rank holds the rows of some chunks; each step, the owner runs the fold
step (its earlier rows plus the chunk itself, causally) and every other rank lets the same
queries attend to what it holds (kvf_attend); ONE exchange - an all-gather of every rank's
normalised output and log-sum-exp, [n, H, d + 1] values per rank - and the merge kernel
(kvf_merge_partials) give the step's output on every rank (row_range_fold_step).

Works on any torch.distributed backend (NCCL on GPUs, gloo on CPU for tests).
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


def max_over_ranks(value: float, device: str | torch.device = "cpu", always: bool = False) -> float:
    """Largest value over the ranks (`always`: run the collective even in a group of one rank)."""
    if not (dist.is_available() and dist.is_initialized()) or (dist.get_world_size() == 1 and not always):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank_step: int, steps: int, world: int, elapsed_ms_max: float) -> float:
    """Aggregate throughput: tokens all ranks folded / the slowest rank's time."""
    return world * steps * tokens_per_rank_step / (elapsed_ms_max * 1e-3)


def chunk_owner(step: int, world: int) -> int:
    """Rank that appends chunk `step` when one sequence's rows are dealt to the ranks chunk by chunk."""
    return step % world


def gather_partials(out: torch.Tensor, lse: torch.Tensor, always: bool = False) -> Tuple[torch.Tensor, torch.Tensor]:
    """All-gather of every rank's (out [n, H, d], lse [n, H]) into ([world, n, H, d], [world, n, H]): the one
    exchange of a step under the row-range split.  Without a process group: the rank's own part, as world 1
    (`always`: run the collective even in a group of one rank)."""
    if not (dist.is_available() and dist.is_initialized()) or (dist.get_world_size() == 1 and not always):
        return out.unsqueeze(0).contiguous(), lse.unsqueeze(0).contiguous()
    world = dist.get_world_size()
    outs = torch.empty((world,) + tuple(out.shape), dtype=out.dtype, device=out.device)
    lses = torch.empty((world,) + tuple(lse.shape), dtype=lse.dtype, device=lse.device)
    # (slices of the two result tensors as the per-rank receive buffers: works on gloo and NCCL alike)
    dist.all_gather(list(outs.unbind(0)), out.contiguous())
    dist.all_gather(list(lses.unbind(0)), lse.contiguous())
    return outs, lses


def row_range_fold_step(cache, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, step: int, pos0: int,
                        rank: int, world: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """One fold step of a sequence whose cache rows are dealt to the ranks chunk by chunk (`cache` is this
    rank's binding.Cache).  Returns the step's (out [n, H, d], lse [n, H]) - the same on every rank."""
    from . import binding
    n, h = q.shape[0], q.shape[1]
    lse = torch.empty((n, h), dtype=torch.float32, device=q.device)
    if chunk_owner(step, world) == rank:
        out = cache.fold_step(q, k, v, pos0=pos0, lse=lse)
    elif len(cache) > 0:
        out = cache.attend(q, pos0=pos0, lse=lse)
    else:
        # nothing held yet: a part that saw no row
        out = torch.zeros((n, h, q.shape[2]), dtype=cache.out_dtype, device=q.device)
        lse.fill_(float("-inf"))
    outs, lses = gather_partials(out, lse)
    return binding.merge_partials(outs, lses)

"""The benchmark's multi-rank plumbing on two gloo ranks (CPU): each rank owns its own sequence,
nothing is exchanged on the data path, elapsed time is reduced with max."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2605_12471_b200 import multi, workloads


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, ret):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    r, wsize, local = multi.env_rank()
    assert (r, wsize, local) == (rank, world, rank)
    w = workloads.TINY
    seq = multi.sequence_of_rank(r)[0]
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, w.tokens, rope_base=w.rope_base)
    outs = []
    for t in range(w.n_steps):
        q, k, v = workloads.chunk_inputs(w, 7, t, sequence=seq)
        outs.append(oc.fold_step(q.double().numpy(), k.double().numpy(), v.double().numpy()))
    checksum = float(np.concatenate(outs).sum())
    fake_ms = 10.0 * (rank + 1)                          # rank 1 is the slow one
    worst = multi.max_over_ranks(fake_ms)
    sums = [None] * world
    dist.all_gather_object(sums, (len(oc), checksum))
    if rank == 0:
        ret["worst"] = worst
        ret["sums"] = sums
        ret["value"] = multi.whole_job_tokens_per_s(w.tokens, 2, world, worst)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_fold_independent_sequences_and_reduce_time_with_max():
    world = 2
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
    assert ret["worst"] == 20.0
    (l0, c0), (l1, c1) = ret["sums"]
    assert l0 == l1 == workloads.TINY.tokens
    assert c0 != c1                                      # different sequences per rank
    assert abs(ret["value"] - 2 * 2 * 512 / 0.020) < 1e-6


def _shard_worker(rank, world, port, ret):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = workloads.Workload("shard_probe", 8, 4, 16, "f32", 8, 40, 10000.0)
    qh, kvh = multi.kv_head_shard(rank, world, w.n_q_heads, w.n_kv_heads)
    oc = oracle.OracleCache(len(qh), len(kvh), w.head_dim, w.tokens, rope_base=w.rope_base)
    outs = []
    for t in range(w.n_steps):
        q, k, v = workloads.chunk_inputs(w, 9, t)                       # every rank draws the same chunk
        qs, ks, vs = multi.shard_heads(q, k, v, rank, world)
        outs.append(oc.fold_step(qs.double().numpy(), ks.double().numpy(), vs.double().numpy()))
    mine = torch.from_numpy(np.concatenate(outs))                       # [T, H / world, d]
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine)                                        # the test's check, not the data path
    if rank == 0:
        ret["out"] = torch.cat(parts, dim=1).numpy()
        ret["heads"] = [(list(a), list(b)) for a, b in
                        (multi.kv_head_shard(r, world, w.n_q_heads, w.n_kv_heads) for r in range(world))]
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_split_one_sequence_by_kv_head_without_any_exchange():
    world = 2
    ret = mp.Manager().dict()
    mp.spawn(_shard_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
    assert ret["heads"] == [([0, 1, 2, 3], [0, 1]), ([4, 5, 6, 7], [2, 3])]
    w = workloads.Workload("shard_probe", 8, 4, 16, "f32", 8, 40, 10000.0)
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, w.tokens, rope_base=w.rope_base)
    full = []
    for t in range(w.n_steps):
        q, k, v = workloads.chunk_inputs(w, 9, t)
        full.append(oc.fold_step(q.double().numpy(), k.double().numpy(), v.double().numpy()))
    assert np.array_equal(ret["out"], np.concatenate(full))             # head slices, nothing else


def test_single_process_helpers():
    assert multi.kv_head_shard(3, 4, 32, 8) == (range(24, 32), range(6, 8))
    import pytest
    with pytest.raises(ValueError):
        multi.kv_head_shard(0, 3, 32, 8)
    assert multi.sequence_of_rank(3, 2) == [6, 7]
    assert multi.max_over_ranks(3.5) == 3.5
    assert multi.whole_job_tokens_per_s(131072, 5, 8, 1000.0) == 8 * 5 * 131072


def _partial(qr, pos_q, rows_k, rows_v, rows_pos, G, scale):
    """Brute-force attention of rotated queries over one rank's rows (numpy): key row j is visible to query i
    iff its position is not later.  Returns (out [n, H, d], lse [n, H]); lse = -inf where nothing is visible."""
    n, H, d = qr.shape
    out = np.zeros((n, H, d))
    lse = np.full((n, H), -np.inf)
    if len(rows_pos) == 0:
        return out, lse
    K, V, pk = np.stack(rows_k), np.stack(rows_v), np.asarray(rows_pos)
    vis = pk[None, :] <= np.asarray(pos_q)[:, None]                       # [n, rows]
    for h in range(H):
        s = (qr[:, h, :] @ K[:, h // G, :].T) * scale
        s = np.where(vis, s, -np.inf)
        m = s.max(axis=1)
        ok = np.isfinite(m)
        p = np.exp(s[ok] - m[ok, None])
        den = p.sum(axis=1)
        out[ok, h, :] = (p / den[:, None]) @ V[:, h // G, :]
        lse[ok, h] = m[ok] + np.log(den)
    return out, lse


def _row_range_worker(rank, world, port, ret):
    from tests import bruteforce
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = workloads.Workload("row_range_probe", 8, 2, 16, "f32", 8, 64, 10000.0)
    G, scale = w.n_q_heads // w.n_kv_heads, 1.0 / np.sqrt(w.head_dim)
    rows_k, rows_v, rows_pos = [], [], []                  # the rows this rank holds (rotated keys, values, positions)
    merged, pos = [], 0
    chunks = [8, 8, 3, 8, 1, 1, 8, 5, 8, 8, 6]
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, 13, t, n_tokens=n)             # every rank draws the same chunk
        p = np.arange(pos, pos + n)
        qr = bruteforce.rope_complex(q.double().numpy(), p, w.rope_base)
        if multi.chunk_owner(t, world) == rank:                            # this rank appends the chunk
            kr = bruteforce.rope_complex(k.double().numpy(), p, w.rope_base)
            rows_k += list(kr); rows_v += list(v.double().numpy()); rows_pos += list(p)
        out, lse = _partial(qr, p, rows_k, rows_v, rows_pos, G, scale)
        outs, lses = multi.gather_partials(torch.from_numpy(out), torch.from_numpy(lse))     # the one exchange
        assert outs.shape == (world, n, w.n_q_heads, w.head_dim) and lses.shape == (world, n, w.n_q_heads)
        o, l = outs.numpy(), lses.numpy()
        tot = np.log(np.exp(l - l.max(axis=0)).sum(axis=0)) + l.max(axis=0)
        merged.append((np.exp(l - tot)[..., None] * o).sum(axis=0))
        pos += n
    if rank == 0:
        ret["merged"] = np.concatenate(merged)
        ret["held"] = len(rows_pos)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_split_one_sequence_by_row_range_with_one_all_gather_per_step():
    """The row-range split on gloo: parts by brute force over each rank's rows, gathered by multi.gather_partials,
    merged by the log-sum-exp weights - equal to the oracle's plain fold of the whole sequence."""
    world = 2
    ret = mp.Manager().dict()
    mp.spawn(_row_range_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
    w = workloads.Workload("row_range_probe", 8, 2, 16, "f32", 8, 64, 10000.0)
    chunks = [8, 8, 3, 8, 1, 1, 8, 5, 8, 8, 6]
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, sum(chunks), rope_base=w.rope_base)
    full = []
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, 13, t, n_tokens=n)
        full.append(oc.fold_step(q.double().numpy(), k.double().numpy(), v.double().numpy()))
    assert ret["held"] == sum(n for t, n in enumerate(chunks) if t % 2 == 0)
    assert np.abs(ret["merged"] - np.concatenate(full)).max() <= 1e-12
    assert [multi.chunk_owner(t, 3) for t in range(5)] == [0, 1, 2, 0, 1]

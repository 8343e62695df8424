"""One sequence split by KV head: each shard folds its heads into its own cache, the outputs are
disjoint head slices and no step needs anything from another shard.  The shards' kernels do not
wait on one another, so they are run one after the other on one GPU here."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_12471_b200 import binding, multi, workloads
from tests.chain import TOL, to_f64

pytestmark = pytest.mark.gpu

W = workloads.Workload("shard_llama_bf16", 32, 8, 128, "bf16", 256, 2048, 500000.0)


@pytest.mark.parametrize("world", [2, 4, 8])
def test_kv_head_shards_reproduce_the_whole_layer(world):
    chunks = [256, 256, 100, 1, 256, 16, 256, 256]
    total = sum(chunks)
    whole = binding.cache_for(W, capacity=total, max_chunk=256)
    shards = []
    for r in range(world):
        qh, kvh = multi.kv_head_shard(r, world, W.n_q_heads, W.n_kv_heads)
        cfg = binding.make_config(len(qh), len(kvh), W.head_dim, "bf16", total, 256, rope_base=W.rope_base)
        shards.append(binding.Cache(cfg))
    oc = oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base)
    worst, worst_pair = 0.0, 0.0
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(W, 81, t, device="cuda", n_tokens=n)
        full = whole.fold_step(q, k, v)
        parts = [shards[r].fold_step(*multi.shard_heads(q, k, v, r, world)) for r in range(world)]
        got = torch.cat(parts, dim=1)                       # head slices side by side: the whole output
        assert got.shape == full.shape
        worst_pair = max(worst_pair, float((got.float() - full.float()).abs().max()))
        rows = sorted({0, n // 2, n - 1})
        ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows)
        worst = max(worst, float(np.abs(to_f64(got[rows]) - ref).max()))
    torch.cuda.synchronize()
    assert all(s.status() == binding.KVF_OK for s in shards)
    assert worst <= TOL["bf16"][0], worst
    assert worst_pair <= 2 ** -5                            # same values up to the order of the partial sums
    # each shard holds exactly its heads' rows: the planes are the whole cache's planes, sliced
    for r in range(world):
        _, kvh = multi.kv_head_shard(r, world, W.n_q_heads, W.n_kv_heads)
        assert torch.equal(shards[r].k_plane()[:, :total], whole.k_plane()[kvh.start:kvh.stop, :total])
        assert torch.equal(shards[r].v_plane()[:, :total], whole.v_plane()[kvh.start:kvh.stop, :total])
